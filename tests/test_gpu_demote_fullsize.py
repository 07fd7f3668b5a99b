"""pw_demote_block at the block shapes of the full-size configurations (14336 x 4096 and 4096 x 14336):
every source -> destination pair against the oracle, bit for bit, and the fifth configuration's protocol on
two full-size layers -- blocks demoted 16 -> 4 -> 2 on a side stream while forward calls run, published
between calls, every demoted page compared with the oracle's chain and one forward call per table epoch
compared with the oracle on sampled tokens."""
import numpy as np
import pytest
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth

from util_gpu import error_metrics, export_to_oracle, make_ctx, pages_equal

pytestmark = pytest.mark.gpu

PAIRS = [(16, 8), (16, 4), (16, 3), (16, 2), (8, 4), (8, 3), (8, 2), (4, 3), (4, 2), (3, 2)]


def test_all_demote_pairs_on_a_full_size_block(orc):
    cfg = synth.CONFIGS["demote_under_load"]
    ctx = make_ctx(synth.CONFIGS["tiny"])
    try:
        w = synth.block_weights(cfg, 0, 0, 0, device="cuda")          # 14336 x 4096
        wh = w.cpu().numpy()
        src_gpu, src_orc = {}, {}
        for sb in (16, 8, 4, 3):
            src_gpu[sb] = ctx.pw_quantize_block(w, sb)
            src_orc[sb] = orc.quantize_block(wh, sb)
        for sb, db in PAIRS:
            got = export_to_oracle(ctx, ctx.pw_demote_block(src_gpu[sb], db), orc)
            ref = orc.demote_block(src_orc[sb], db)
            assert pages_equal(got, ref), (sb, db)
            del got, ref
    finally:
        ctx.close()


def test_down_shaped_full_size_block_chain(orc):
    cfg = synth.CONFIGS["demote_under_load"]
    ctx = make_ctx(synth.CONFIGS["tiny"])
    try:
        w = synth.block_weights(cfg, 1, 5, 2, device="cuda")          # 4096 x 14336
        p4 = ctx.pw_demote_block(ctx.pw_quantize_block(w, 16), 4)
        p2 = ctx.pw_demote_block(p4, 2)
        r4 = orc.demote_block(orc.quantize_block(w.cpu().numpy(), 16), 4)
        assert pages_equal(export_to_oracle(ctx, p4, orc), r4)
        assert pages_equal(export_to_oracle(ctx, p2, orc), orc.demote_block(r4, 2))
    finally:
        ctx.close()


def test_demote_under_load_on_full_size_layers(orc):
    cfg = synth.CONFIGS["demote_under_load"]
    L, T, k, E = 2, cfg.tokens, cfg.top_k, cfg.n_experts
    ctx = B.Context(L, E, 0, cfg.hidden, cfg.ffn, T, k)
    try:
        pages, opages = {}, {}
        for l in range(L):
            ents = []
            for e in range(E):
                for u in range(3):
                    w = synth.block_weights(cfg, l, e, u, device="cuda")
                    pages[(l, e, u)] = ctx.pw_quantize_block(w, 16)
                    opages[(l, e, u)] = orc.quantize_block(w.cpu().numpy(), 16)
                    ents.append((l, e, u, pages[(l, e, u)]))
                    del w
            ctx.pw_set_page_table(ents)
        xs = [synth.activations(cfg, l, device="cuda") for l in range(L)]
        lgs = [synth.router_logits(cfg, l, device="cuda") for l in range(L)]
        # a seeded handful of the schedule's blocks that covers both block shapes
        sched = [key for key in synth.demote_schedule(cfg) if key[0] < L]
        picked = [key for key in sched if key[2] == 2][:3] + [key for key in sched if key[2] != 2][:4]
        assert len(picked) == 7
        rng = np.random.default_rng(7)
        toks = sorted(rng.choice(T, size=4, replace=False).tolist())
        main, side = torch.cuda.current_stream(), torch.cuda.Stream()
        keep_alive, checks = [], []

        def snapshot(layer):
            out = ctx.pw_moe_forward(layer, xs[layer], lgs[layer], k)
            checks.append((layer, out.clone(), [opages[(layer, e, u)] for e in range(E) for u in range(3)]))

        for l in range(L):
            snapshot(l)                                       # epoch 0: all 16-bit
        step = 0
        for dst_bits in (4, 2):
            side.wait_stream(main)
            inflight = []
            for key in picked:
                new = ctx.pw_demote_block(pages[key], dst_bits, stream=side)
                ev = torch.cuda.Event()
                ev.record(side)
                inflight.append((key, new, ev))
                for _ in range(3):                           # forward calls keep running under the demote
                    ctx.pw_moe_forward(step % L, xs[step % L], lgs[step % L], k)
                    step += 1
                done = [x for x in inflight if x[2].query()]
                if done:
                    for kk, pg, ev2 in done:
                        main.wait_event(ev2)
                        keep_alive.append(pages[kk])
                        pages[kk] = pg
                        opages[kk] = orc.demote_block(opages[kk], dst_bits)
                    ctx.pw_set_page_table([(kk[0], kk[1], kk[2], pg) for kk, pg, _ in done])
                    inflight = [x for x in inflight if not any(x is d for d in done)]
            for kk, pg, ev2 in inflight:
                ev2.synchronize()
                keep_alive.append(pages[kk])
                pages[kk] = pg
                opages[kk] = orc.demote_block(opages[kk], dst_bits)
            if inflight:
                ctx.pw_set_page_table([(kk[0], kk[1], kk[2], pg) for kk, pg, _ in inflight])
            for l in range(L):
                snapshot(l)                                   # one forward call of this epoch per layer
        torch.cuda.synchronize()
        assert ctx.pw_last_device_status() == 0
        for key in picked:
            assert pages[key].bits == 2
            assert pages_equal(export_to_oracle(ctx, pages[key], orc), opages[key]), key
        for layer, out, snap in checks:
            ref = orc.moe_forward(xs[layer].cpu().numpy(), lgs[layer].cpu().numpy(), k, snap, tokens=toks)
            max_abs, rel_f = error_metrics(out.cpu().numpy()[toks], ref[toks])
            assert max_abs <= 2e-2 and rel_f <= 5e-3, (layer, max_abs, rel_f)
    finally:
        ctx.close()
