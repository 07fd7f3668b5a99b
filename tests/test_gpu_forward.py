"""GPU parity of pw_moe_forward against the oracle: routing bit-exact, outputs within tolerance."""
import numpy as np
import pytest
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth

from util_gpu import build_layer, error_metrics, export_to_oracle, import_from_oracle, make_ctx

pytestmark = pytest.mark.gpu

MAX_ABS, REL_F = 2e-2, 5e-3          # tolerance of the layer output (fp16 operands, fp32 accumulate)
MODES = [B.PW_MODE_SIMT, B.PW_MODE_TENSOR]


def check_routing(ctx, orc, logits, T, k, E):
    r = {n: v.cpu().numpy() for n, v in ctx.pw_get_routing(T, k).items()}
    ids, gates = orc.router(logits, k)
    counts, offsets, perm, _ = orc.permute(ids, E)
    assert np.array_equal(r["topk_ids"], ids)
    assert np.array_equal(r["counts"], counts)
    assert np.array_equal(r["offsets"], offsets)
    assert np.array_equal(r["perm"], perm)
    assert np.allclose(r["gates"], gates, rtol=1e-6, atol=1e-9)


def run_case(orc, cfg, mode, tokens=None, bits=None, sample_tokens=None):
    T = tokens or cfg.tokens
    ctx = make_ctx(cfg, max_tokens=T, n_layers=1)
    try:
        pages, bits = build_layer(ctx, cfg, 0, bits)
        x = synth.activations(cfg, device="cuda", tokens=T)
        logits = synth.router_logits(cfg, device="cuda", tokens=T)
        out = ctx.pw_moe_forward(0, x, logits, cfg.top_k, mode=mode)
        torch.cuda.synchronize()
        assert ctx.pw_last_device_status() == 0
        check_routing(ctx, orc, logits.cpu().numpy(), T, cfg.top_k, cfg.n_experts)
        opages = [export_to_oracle(ctx, p, orc) for p in pages]
        ref = orc.moe_forward(x.cpu().numpy(), logits.cpu().numpy(), cfg.top_k, opages, n_shared=cfg.n_shared,
                              tokens=sample_tokens)
        got = out.cpu().numpy()
        if sample_tokens is not None:
            got, ref = got[sample_tokens], ref[sample_tokens]
        assert np.isfinite(got).all()
        max_abs, rel_f = error_metrics(got, ref)
        assert max_abs <= MAX_ABS and rel_f <= REL_F, (max_abs, rel_f)
        return max_abs, rel_f
    finally:
        ctx.close()


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("name", ["tiny", "tiny_cover"])
def test_tiny_configs(orc, name, mode):
    run_case(orc, synth.CONFIGS[name], mode)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("bits", [16, 8, 4, 3, 2])
def test_uniform_bitwidth_table(orc, bits, mode):
    cfg = synth.CONFIGS["tiny"]
    run_case(orc, cfg, mode, bits=np.full((8, 3), bits, np.int32))


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("T", [1, 3, 17, 130])
def test_ragged_token_counts(orc, T, mode):
    run_case(orc, synth.CONFIGS["tiny_cover"], mode, tokens=T)


@pytest.mark.parametrize("mode", MODES)
def test_shared_experts_and_many_experts(orc, mode):
    cfg = synth.LayerConfig("fg_small", 64, 6, 256, 384, 96, n_shared=2, routing="zipf", zipf_a=1.2,
                            bit_rule="int4_10fp16_20int2")
    run_case(orc, cfg, mode)


@pytest.mark.parametrize("mode", MODES)
def test_gate_and_up_sharing_one_bitwidth(orc, mode):
    # the paper's block types are {gate_up, down}: gate and up of an expert always at the same bitwidth
    cfg = synth.CONFIGS["tiny"]
    rng = np.random.default_rng(3)
    gu = rng.choice(synth.BITS, size=8)
    dn = rng.choice(synth.BITS, size=8)
    run_case(orc, cfg, mode, bits=np.stack([gu, gu, dn], axis=1).astype(np.int32))


def test_forward_from_imported_oracle_pages(orc):
    cfg = synth.CONFIGS["tiny_cover"]
    ctx = make_ctx(cfg, n_layers=1)
    bits = synth.assign_bits(cfg)
    opages, entries, keep = [], [], []
    for e in range(8):
        for u in range(3):
            op = orc.quantize_block(synth.block_weights(cfg, 0, e, u).numpy(), int(bits[e, u]))
            opages.append(op)
            keep.append(import_from_oracle(ctx, op))
            entries.append((0, e, u, keep[-1]))
    ctx.pw_set_page_table(entries)
    x = synth.activations(cfg, device="cuda")
    logits = synth.router_logits(cfg, device="cuda")
    out = ctx.pw_moe_forward(0, x, logits, cfg.top_k, mode=B.PW_MODE_SIMT).cpu().numpy()
    ref = orc.moe_forward(x.cpu().numpy(), logits.cpu().numpy(), cfg.top_k, opages)
    max_abs, rel_f = error_metrics(out, ref)
    assert max_abs <= MAX_ABS and rel_f <= REL_F
    ctx.close()


def test_router_ties_follow_the_index_rule(orc):
    cfg = synth.CONFIGS["tiny"]
    ctx = make_ctx(cfg, max_tokens=64, n_layers=1)
    pages, _ = build_layer(ctx, cfg, 0, np.full((8, 3), 4, np.int32))
    x = synth.activations(cfg, device="cuda", tokens=64)
    logits = torch.round(synth.router_logits(cfg, device="cuda", tokens=64) * 2) / 2     # many exact ties
    logits[0] = 0.0
    ctx.pw_moe_forward(0, x, logits.contiguous(), 2, mode=B.PW_MODE_SIMT)
    check_routing(ctx, orc, logits.cpu().numpy(), 64, 2, 8)
    ctx.close()


def test_commit_is_stream_ordered_and_forward_reads_the_committed_row(orc):
    # demote one block, publish it between two forward calls: the first call sees the old page,
    # the second the new one, and tokens not routed to that expert do not change
    cfg = synth.CONFIGS["tiny"]
    ctx = make_ctx(cfg, n_layers=1)
    pages, bits = build_layer(ctx, cfg, 0, np.full((8, 3), 8, np.int32))
    x = synth.activations(cfg, device="cuda")
    logits = synth.router_logits(cfg, device="cuda")
    e0 = ctx.pw_set_page_table([])
    out_a = ctx.pw_moe_forward(0, x, logits, 2, mode=B.PW_MODE_SIMT)
    side = torch.cuda.Stream()
    low = ctx.pw_demote_block(pages[3 * 5 + 2], 2, stream=side)          # expert 5, down, 8 -> 2 on a side stream
    done = torch.cuda.Event()
    done.record(side)
    out_b = ctx.pw_moe_forward(0, x, logits, 2, mode=B.PW_MODE_SIMT)     # still the old row
    torch.cuda.current_stream().wait_event(done)
    e1 = ctx.pw_set_page_table([(0, 5, 2, low)])
    out_c = ctx.pw_moe_forward(0, x, logits, 2, mode=B.PW_MODE_SIMT)
    torch.cuda.synchronize()
    assert e1 == e0 + 1
    assert ctx.pw_query_row(0, 5, 2).page.bits == 2
    assert torch.equal(out_a, out_b)
    ids, _ = orc.router(logits.cpu().numpy(), 2)
    hit = torch.from_numpy((ids == 5).any(axis=1)).cuda()
    assert hit.any() and (~hit).any()
    assert torch.equal(out_a[~hit], out_c[~hit])
    assert (out_a[hit] != out_c[hit]).any(dim=1).all()
    opages = [export_to_oracle(ctx, p, orc) for p in pages]
    opages[3 * 5 + 2] = export_to_oracle(ctx, low, orc)
    ref = orc.moe_forward(x.cpu().numpy(), logits.cpu().numpy(), 2, opages)
    max_abs, rel_f = error_metrics(out_c.cpu().numpy(), ref)
    assert max_abs <= MAX_ABS and rel_f <= REL_F
    ctx.close()


def test_forward_argument_errors(orc):
    cfg = synth.CONFIGS["tiny"]
    ctx = make_ctx(cfg, n_layers=2)
    x = synth.activations(cfg, device="cuda")
    logits = synth.router_logits(cfg, device="cuda")
    with pytest.raises(B.PwError) as e:
        ctx.pw_moe_forward(0, x, logits, 2)               # nothing published yet
    assert e.value.status == 5
    pages, _ = build_layer(ctx, cfg, 0)
    with pytest.raises(B.PwError) as e:
        ctx.pw_moe_forward(1, x, logits, 2)               # layer 1 still unpublished
    assert e.value.status == 5
    for bad_k in (0, 3, 9):
        with pytest.raises(B.PwError) as e:
            ctx.pw_moe_forward(0, x, logits, bad_k)
        assert e.value.status == 1
    big = torch.zeros(17, 256, dtype=torch.float16, device="cuda")
    with pytest.raises(B.PwError) as e:
        ctx.pw_moe_forward(0, big, torch.zeros(17, 8, device="cuda"), 2)
    assert e.value.status == 1
    wrong = B.Page(512, 256, 4)                           # a gate-shaped page offered as a down block
    with pytest.raises(B.PwError) as e:
        ctx.pw_set_page_table([(0, 0, 2, wrong)])
    assert e.value.status == 2
    can = ctx.pw_export_page(pages[0])
    with pytest.raises(B.PwError) as e:
        ctx.pw_set_page_table([(0, 0, 0, can)])           # canonical layout cannot be published
    assert e.value.status == 5
    with pytest.raises(B.PwError) as e:
        ctx.pw_set_page_table([(0, 0, 0, pages[0])], state=B.PW_STATE_CPU_RESIDENT)
    assert e.value.status == 5
    assert ctx.pw_last_device_status() == 0
    ctx.close()


@pytest.mark.parametrize("mode", MODES)
def test_forward_is_bitwise_reproducible(mode):
    """CTAs claim units in whatever order they finish, but every output element is accumulated by one issuer
    per K range in a fixed order, the partials and splits are added in a fixed order, and the combine walks
    the slots in order: repeated calls return the same bits."""
    cfg = synth.CONFIGS["tiny_cover"]
    T = 48
    ctx = make_ctx(cfg, max_tokens=T, n_layers=1)
    try:
        pages, _ = build_layer(ctx, cfg, 0, None)
        x = synth.activations(cfg, device="cuda", tokens=T)
        logits = synth.router_logits(cfg, device="cuda", tokens=T)
        first = ctx.pw_moe_forward(0, x, logits, cfg.top_k, mode=mode).clone()
        for _ in range(5):
            again = ctx.pw_moe_forward(0, x, logits, cfg.top_k, mode=mode)
            torch.cuda.synchronize()
            assert torch.equal(first.view(torch.int32), again.view(torch.int32))
        assert ctx.pw_last_device_status() == 0
    finally:
        ctx.close()


def test_forward_repeats_bit_for_bit_when_the_tile_counts_are_odd():
    """More units than CTAs, so the later units are claimed in an order that changes from run to run, and odd
    numbers of K tiles per unit (3 for gate/up, 5 for down), so a unit's first tile falls on a different
    partial accumulator depending on what its CTA ran before: the partials are added starting from the one
    that holds the unit's first tile, and the result does not depend on that history."""
    cfg = synth.LayerConfig("odd_tiles", 96, 6, 384, 640, 64, n_shared=1, routing="normal", bit_rule="iid5")
    ctx = make_ctx(cfg, max_tokens=cfg.tokens, n_layers=1)
    try:
        build_layer(ctx, cfg, 0, None)
        x = synth.activations(cfg, device="cuda")
        logits = synth.router_logits(cfg, device="cuda")
        first = ctx.pw_moe_forward(0, x, logits, cfg.top_k).clone()
        side = torch.cuda.Stream()
        for i in range(60):
            if i % 5 == 0:
                with torch.cuda.stream(side):        # other work on the device shifts which CTA finishes first
                    torch.cuda._sleep(100000)
            again = ctx.pw_moe_forward(0, x, logits, cfg.top_k)
            assert torch.equal(first.view(torch.int32), again.view(torch.int32)), i
        torch.cuda.synchronize()
        assert ctx.pw_last_device_status() == 0
    finally:
        ctx.close()


def test_many_calls_with_wide_token_tiles_on_short_units(orc):
    """Short contractions (4 K-tiles per gate/up unit, 16 per down unit), several units per CTA, token tiles wider than 32: the kernels
    whose wide units share accumulators, two issuers taking turns on each.  One issuer is regularly a unit ahead
    of the other at a unit boundary; the turn word must survive that (an earlier version lost a turn there and
    ran into its bounded waits once in a few hundred units).  Several hundred calls over three layers of mixed
    pages, every call checked against the first of its layer bit for bit, one of them against the oracle."""
    cfg = synth.LayerConfig("wide_short", 16, 2, 512, 2048, 512, routing="normal", bit_rule="iid5", n_layers=3)
    ctx = make_ctx(cfg, max_tokens=cfg.tokens, n_layers=3)
    try:
        pages = [build_layer(ctx, cfg, l, None)[0] for l in range(3)]
        x = synth.activations(cfg, device="cuda")
        logits = synth.router_logits(cfg, device="cuda")
        first = [ctx.pw_moe_forward(l, x, logits, cfg.top_k).clone() for l in range(3)]
        counts = ctx.pw_get_routing(cfg.tokens, cfg.top_k)["counts"].cpu().numpy()
        assert counts.min() > 32                              # every expert takes wide token tiles
        for i in range(450):
            l = i % 3
            again = ctx.pw_moe_forward(l, x, logits, cfg.top_k)
            if i % 50 == 0:
                assert ctx.pw_last_device_status() == 0, i
            assert torch.equal(first[l].view(torch.int32), again.view(torch.int32)), i
        torch.cuda.synchronize()
        assert ctx.pw_last_device_status() == 0
        opages = [export_to_oracle(ctx, p, orc) for p in pages[1]]
        sample = list(range(0, cfg.tokens, 16))
        ref = orc.moe_forward(x.cpu().numpy(), logits.cpu().numpy(), cfg.top_k, opages, tokens=sample)
        max_abs, rel_f = error_metrics(first[1].cpu().numpy()[sample], ref[sample])
        assert max_abs <= MAX_ABS and rel_f <= REL_F, (max_abs, rel_f)
    finally:
        ctx.close()


def test_back_to_back_calls_with_different_routing(orc):
    """Consecutive calls reuse the workspace (unit lists, counters, operand buffers) while the kernels of the
    call before may still be draining: alternate two token sets and check every result against the oracle."""
    cfg = synth.CONFIGS["tiny_cover"]
    ctx = make_ctx(cfg, max_tokens=cfg.tokens, n_layers=1)
    try:
        pages, _ = build_layer(ctx, cfg, 0, None)
        opages = [export_to_oracle(ctx, p, orc) for p in pages]
        sets = []
        for step in range(2):
            x = synth.activations(cfg, step=step, device="cuda")
            logits = synth.router_logits(cfg, step=step, device="cuda")
            ref = orc.moe_forward(x.cpu().numpy(), logits.cpu().numpy(), cfg.top_k, opages, n_shared=cfg.n_shared)
            sets.append((x, logits, ref))
        outs = []
        for i in range(8):                                   # enqueue all calls first, read back afterwards
            x, logits, _ = sets[i % 2]
            outs.append(ctx.pw_moe_forward(0, x, logits, cfg.top_k, mode=B.PW_MODE_TENSOR).clone())
        torch.cuda.synchronize()
        assert ctx.pw_last_device_status() == 0
        for i, out in enumerate(outs):
            max_abs, rel_f = error_metrics(out.cpu().numpy(), sets[i % 2][2])
            assert max_abs <= MAX_ABS and rel_f <= REL_F, (i, max_abs, rel_f)
    finally:
        ctx.close()


@pytest.mark.parametrize("tokens", [600, 1100])
def test_wide_and_narrow_token_tiles_together(orc, tokens):
    """Enough tokens per expert for 128-token tiles (the kernel variant whose issuer warps share the epilogue),
    with remainders that make narrow, double-buffered units in the same launch."""
    run_case(orc, synth.CONFIGS["tiny_cover"], B.PW_MODE_TENSOR, tokens=tokens)


def test_forward_call_replays_from_a_cuda_graph(orc):
    """A layer call is six dependent launches; captured once into a CUDA graph it replays on new contents of
    the same buffers (what a launch-bound decode loop does) and returns the bits of the eager call."""
    cfg = synth.CONFIGS["tiny_cover"]
    ctx = make_ctx(cfg, n_layers=1)
    try:
        pages, _ = build_layer(ctx, cfg, 0, None)
        xs = [synth.activations(cfg, step=s, device="cuda") for s in range(3)]
        lgs = [synth.router_logits(cfg, step=s, device="cuda") for s in range(3)]
        eager = [ctx.pw_moe_forward(0, xs[s], lgs[s], cfg.top_k).clone() for s in range(3)]   # also sets the kernels up
        x, lg = xs[0].clone(), lgs[0].clone()
        out = torch.empty(cfg.tokens, cfg.hidden, dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            ctx.pw_moe_forward(0, x, lg, cfg.top_k, out=out)
        for s in (1, 2, 0, 2):
            x.copy_(xs[s])
            lg.copy_(lgs[s])
            graph.replay()
            torch.cuda.synchronize()
            assert torch.equal(out, eager[s]), s
        assert ctx.pw_last_device_status() == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("shape", [(256, 32, 16, 128, 128, 40),     # the most experts, choices and shared experts a context takes
                                   (4, 4, 0, 128, 256, 19),          # every expert chosen by every token
                                   (1, 1, 0, 256, 128, 5)])          # a single expert
def test_limits_of_the_configuration(orc, shape, mode):
    E, k, n_shared, H, F, T = shape
    cfg = synth.LayerConfig("limits_%d_%d" % (E, k), E, k, H, F, T, n_shared=n_shared, routing="normal", bit_rule="iid5")
    run_case(orc, cfg, mode)


def test_host_buffer_entry_point_matches_the_device_one(orc):
    """pw_moe_forward_host stages the inputs, runs the same kernels and copies the result back, ordered on the
    stream: same bits as the device call, with pinned and with pageable host buffers, several calls in a row."""
    cfg = synth.CONFIGS["tiny_cover"]
    ctx = make_ctx(cfg, n_layers=1)
    try:
        pages, _ = build_layer(ctx, cfg, 0, None)
        for step, pinned in ((0, True), (1, False), (2, True)):
            x = synth.activations(cfg, step=step, device="cuda")
            lg = synth.router_logits(cfg, step=step, device="cuda")
            want = ctx.pw_moe_forward(0, x, lg, cfg.top_k).clone()
            xh, lh = x.cpu(), lg.cpu()
            oh = torch.empty(cfg.tokens, cfg.hidden, dtype=torch.float32)
            if pinned:
                xh, lh, oh = xh.pin_memory(), lh.pin_memory(), oh.pin_memory()
            ctx.pw_moe_forward_host(0, xh, lh, cfg.top_k, oh)
            torch.cuda.synchronize()
            assert torch.equal(oh, want.cpu()), (step, pinned)
        with pytest.raises(B.PwError) as e:
            big = torch.zeros(cfg.tokens + 1, cfg.hidden, dtype=torch.float16)
            ctx.pw_moe_forward_host(0, big, torch.zeros(cfg.tokens + 1, cfg.n_experts), cfg.top_k,
                                    torch.empty(cfg.tokens + 1, cfg.hidden))
        assert e.value.status == 1
        # an argument error is found before any copy is enqueued: nothing is launched, the staging buffers keep
        # the previous call's inputs (the next device-side call on them gives the previous result)
        n0 = ctx.pw_launch_count()
        junk = torch.full((cfg.tokens, cfg.hidden), 7.0, dtype=torch.float16)
        with pytest.raises(B.PwError) as e:
            ctx.pw_moe_forward_host(0, junk, lh, cfg.n_experts + 1, oh)       # top_k out of range
        assert e.value.status == 1 and ctx.pw_launch_count() == n0
        torch.cuda.synchronize()
        ctx.pw_moe_forward_host(0, xh, lh, cfg.top_k, oh)
        torch.cuda.synchronize()
        assert torch.equal(oh, want.cpu())
        assert ctx.pw_last_device_status() == 0
    finally:
        ctx.close()
