"""The whole loop on the GPU: observation taps -> planner -> demote, commit, offload -> forward, against the
oracle carrying out the same plan."""
import numpy as np
import pytest
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth

from util_gpu import build_layer, error_metrics, export_to_oracle, make_ctx

pytestmark = pytest.mark.gpu

LEVELS = (16, 8, 4, 3, 2)


def test_taps_planner_demote_offload_forward(orc):
    cfg = synth.CONFIGS["tiny"]
    E, S = cfg.n_experts, cfg.n_experts
    ctx = make_ctx(cfg, n_layers=1)
    try:
        bits = np.full((S, 3), 16, np.int32)
        pages, _ = build_layer(ctx, cfg, 0, bits)
        opages = [export_to_oracle(ctx, p, orc) for p in pages]
        x = synth.activations(cfg, device="cuda")
        lg = synth.router_logits(cfg, device="cuda")
        ctx.pw_observe(True)
        ctx.pw_moe_forward(0, x, lg, cfg.top_k)
        mass, phi = ctx.pw_observation_summary(0)
        ctx.pw_observe(False)
        torch.cuda.synchronize()
        mass, phi = mass.cpu().numpy()[None], phi.cpu().numpy()[None]

        # tables: every block exists at every level; sensitivities grow as the bitwidth falls (seeded stand-ins)
        rng = np.random.default_rng(11)
        sens = np.sort(rng.random((1, S, 3, 5)).astype(np.float32), axis=-1)
        nbytes = np.zeros((1, S, 3, 5), np.uint64)
        for u in range(3):
            rows, cols = cfg.block_shape(u)
            for lv, b in enumerate(LEVELS):
                nbytes[0, :, u, lv] = B.pw_page_bytes(rows, cols, b)[0]
        target = B.pw_kv_pressure_bytes(4, 1, int(nbytes[0, 0, 0, 0]))        # four blocks' worth of 16-bit pages
        steps, released, stage = B.pw_plan_step(1, E, 0, bits.astype(np.uint8)[None], np.ones((1, S, 3, 5), np.uint8),
                                                sens, nbytes, mass, [0.25, 1.0], [8.0, 1.0], [[8, 2]], target, phi=phi)
        assert released >= target and stage == 0 and len(steps) > 0
        hot = int(np.argmax(mass[0]))
        assert all(b2 >= 8 for (l, e, u, b, b2, d) in steps if e == hot)      # the hottest expert keeps 8 bits

        # carry the plan out: demote on a side stream, commit, then move the page that is no longer needed out
        side = torch.cuda.Stream()
        before = sum(B.pw_page_bytes(p.rows, p.cols, p.bits)[0] for p in pages)
        hosts = []
        for (l, e, u, b, b2, d) in steps:
            old = pages[e * 3 + u]
            assert old.bits == b
            side.wait_stream(torch.cuda.current_stream())
            new = ctx.pw_demote_block(old, b2, stream=side)
            torch.cuda.current_stream().wait_stream(side)
            ctx.pw_set_page_table([(0, e, u, new)])
            hosts.append(ctx.pw_offload_page(0, e, u, old, stream=side))
            pages[e * 3 + u] = new
            opages[e * 3 + u] = orc.demote_block(opages[e * 3 + u], b2)
        side.synchronize()
        after = sum(B.pw_page_bytes(p.rows, p.cols, p.bits)[0] for p in pages)
        assert before - after == released
        for (l, e, u, b, b2, d) in steps:
            assert ctx.pw_page_state(0, e, u, b) == B.PW_STATE_CPU_RESIDENT
        assert ctx.pw_query_row(0, steps[-1][1], steps[-1][2]).page.bits == steps[-1][4]

        out = ctx.pw_moe_forward(0, x, lg, cfg.top_k).cpu().numpy()
        assert ctx.pw_last_device_status() == 0
        ref = orc.moe_forward(x.cpu().numpy(), lg.cpu().numpy(), cfg.top_k, opages)
        max_abs, rel_f = error_metrics(out, ref)
        assert max_abs <= 2e-2 and rel_f <= 5e-3
    finally:
        ctx.close()


def test_taps_planner_plane_movement_forward(orc):
    """The same loop on a layer whose blocks are overlaid bit-planes: a step of the plan is carried out by
    publishing the block at the lower bitwidth (no kernel) and moving the plane it no longer reads to the host."""
    from oracle import planes as PL
    cfg = synth.CONFIGS["tiny"]
    E, S = cfg.n_experts, cfg.n_experts
    ctx = make_ctx(cfg, n_layers=1)
    try:
        blocks, refs, entries = [], [], []
        for e in range(S):
            for u in range(3):
                w = synth.block_weights(cfg, 0, e, u, device="cuda")
                blocks.append(ctx.pw_quantize_planes(w))
                refs.append(PL.quantize_planes(w.cpu().numpy()))
                entries.append((0, e, u, blocks[-1].at(4)))
        ctx.pw_set_page_table(entries)
        q = np.full((S, 3), 4, np.int32)
        x = synth.activations(cfg, device="cuda")
        lg = synth.router_logits(cfg, device="cuda")
        ctx.pw_observe(True)
        ctx.pw_moe_forward(0, x, lg, cfg.top_k)
        mass, phi = ctx.pw_observation_summary(0)
        ctx.pw_observe(False)
        torch.cuda.synchronize()
        mass, phi = mass.cpu().numpy()[None], phi.cpu().numpy()[None]

        # a bit-plane block supports 4, 3 and 2 bits; the size table is Eq. 3's (planes read + one table state)
        rng = np.random.default_rng(5)
        sens = np.sort(rng.random((1, S, 3, 5)).astype(np.float32), axis=-1)
        supported = np.zeros((1, S, 3, 5), np.uint8)
        supported[..., 2:] = 1
        nbytes = np.zeros((1, S, 3, 5), np.uint64)
        for u in range(3):
            rows, cols = cfg.block_shape(u)
            for lv, b in enumerate(LEVELS):
                nbytes[0, :, u, lv] = B.pw_page_bytes(rows, cols, b)[0]
        plane_bytes = {u: B.pw_plane_bytes(*cfg.block_shape(u))[2] for u in range(3)}
        target = 10 * plane_bytes[0]
        steps, released, stage = B.pw_plan_step(1, E, 0, q.astype(np.uint8)[None], supported, sens, nbytes, mass,
                                                [0.25, 1.0], [8.0, 1.0], [[3, 2]], target, phi=phi)
        assert released >= target and len(steps) > 0
        hot = int(np.argmax(mass[0]))
        assert all(b2 >= 3 for (l, e, u, b, b2, d) in steps if e == hot)      # the hottest expert keeps 3 bits

        side = torch.cuda.Stream()
        n0 = ctx.pw_launch_count()
        moved = 0
        for (l, e, u, b, b2, d) in steps:
            assert q[e, u] == b and b2 == b - 1
            ctx.pw_set_page_table([(0, e, u, blocks[e * 3 + u].at(b2))])       # lower q_i first ...
            side.wait_stream(torch.cuda.current_stream())
            ctx.pw_offload_plane(0, e, u, blocks[e * 3 + u], b, stream=side)  # ... then plane b moves out
            moved += plane_bytes[u]
            q[e, u] = b2
        assert ctx.pw_launch_count() - n0 == len(steps)                        # the commits; no page is rewritten
        assert moved == released                                               # Eq. 3: a plane per step
        side.synchronize()
        for (l, e, u, b, b2, d) in steps:
            assert ctx.pw_plane_state(0, e, u, b) == B.PW_STATE_CPU_RESIDENT

        out = ctx.pw_moe_forward(0, x, lg, cfg.top_k).cpu().numpy()
        assert ctx.pw_last_device_status() == 0
        views = [PL.view(refs[e * 3 + u], int(q[e, u])) for e in range(S) for u in range(3)]
        ref = orc.moe_forward(x.cpu().numpy(), lg.cpu().numpy(), cfg.top_k, views)
        max_abs, rel_f = error_metrics(out, ref)
        assert max_abs <= 2e-2 and rel_f <= 5e-3
    finally:
        ctx.close()
