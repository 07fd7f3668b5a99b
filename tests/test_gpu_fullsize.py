"""Full-size configurations in the launch configuration the benchmark times (mode AUTO): routing
and permutation bit-exact on every token, layer outputs compared on sampled tokens the oracle
computes one by one, pages compared bit for bit on sampled blocks."""
import numpy as np
import pytest
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth

from util_gpu import build_layer, error_metrics, export_to_oracle, make_ctx, pages_equal

pytestmark = pytest.mark.gpu

MAX_ABS, REL_F = 2e-2, 5e-3


def full_case(orc, name, n_sample, check_blocks):
    cfg = synth.CONFIGS[name]
    ctx = make_ctx(cfg, n_layers=1)
    try:
        pages, bits = build_layer(ctx, cfg, 0)
        x = synth.activations(cfg, device="cuda")
        logits = synth.router_logits(cfg, device="cuda")
        out = ctx.pw_moe_forward(0, x, logits, cfg.top_k, mode=B.PW_MODE_AUTO)
        torch.cuda.synchronize()
        assert ctx.pw_last_device_status() == 0
        T, k, E = cfg.tokens, cfg.top_k, cfg.n_experts
        r = {n: v.cpu().numpy() for n, v in ctx.pw_get_routing(T, k).items()}
        lg = logits.cpu().numpy()
        ids, gates = orc.router(lg, k)
        counts, offsets, perm, _ = orc.permute(ids, E)
        assert np.array_equal(r["topk_ids"], ids) and np.array_equal(r["counts"], counts)
        assert np.array_equal(r["offsets"], offsets) and np.array_equal(r["perm"], perm)
        assert np.allclose(r["gates"], gates, rtol=1e-6, atol=1e-9)
        # sampled blocks: the GPU quantizer against the oracle's, bit for bit
        for (e, u) in check_blocks:
            w = synth.block_weights(cfg, 0, e, u, device="cuda")
            ref = orc.quantize_block(w.cpu().numpy(), int(bits[e, u]))
            assert pages_equal(export_to_oracle(ctx, pages[e * 3 + u], orc), ref), (e, u)
        rng = np.random.default_rng(1)
        toks = sorted(rng.choice(T, size=min(n_sample, T), replace=False).tolist())
        opages = [export_to_oracle(ctx, p, orc) for p in pages]
        ref = orc.moe_forward(x.cpu().numpy(), lg, k, opages, n_shared=cfg.n_shared, tokens=toks)
        got = out.cpu().numpy()
        assert np.isfinite(got).all()
        max_abs, rel_f = error_metrics(got[toks], ref[toks])
        assert max_abs <= MAX_ABS and rel_f <= REL_F, (max_abs, rel_f)
    finally:
        ctx.close()


def test_mixtral_decode_full_size(orc):
    full_case(orc, "mixtral_decode", 12, [(0, 0), (3, 2)])


def test_finegrained_decode_full_size(orc):
    full_case(orc, "finegrained_decode", 48, [(0, 0), (17, 1), (40, 2), (65, 2)])


def test_mixtral_prefill_full_size(orc):
    full_case(orc, "mixtral_prefill", 8, [(5, 1)])


@pytest.mark.parametrize("name", ["latency_b1", "latency_b4"])
def test_latency_decode_full_size(orc, name):
    # batch 1 and batch 4 on the 60 + 4 expert layer: every token is checked
    full_case(orc, name, 4, [(0, 0), (33, 2), (61, 1)])


def test_manyexpert_decode_full_size(orc):
    full_case(orc, "manyexpert_decode", 24, [(0, 0), (77, 1), (128, 2)])
