"""pw_route_tokens_static: the routing entry point for callers that cannot allocate device memory
(no context, no workspace; scratch lives in a fixed array inside the library).  Checked against the
routing that pw_moe_forward performs and against the CPU oracle's router and stable permutation, on two
calls in a row, since every call reuses the same scratch."""
import numpy as np
import pytest
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth

from util_gpu import build_layer, make_ctx

pytestmark = pytest.mark.gpu


def reference_routing(cfg, logits, T):
    ctx = make_ctx(cfg, max_tokens=T, n_layers=1)
    pages, _ = build_layer(ctx, cfg, 0, np.full((cfg.n_experts + cfg.n_shared, 3), 16, np.int32))
    x = synth.activations(cfg, device="cuda", tokens=T)
    ctx.pw_moe_forward(0, x, logits, cfg.top_k)
    r = {k: v.clone() for k, v in ctx.pw_get_routing(T, cfg.top_k).items()}
    torch.cuda.synchronize()
    ctx.close()
    return r


def check_against_oracle(orc, got, logits, top_k):
    """Indices bit for bit, gates to 1e-6 relative (expf differs by ulps between libm and the device)."""
    lg = logits.cpu().numpy()
    ids, gates = orc.router(lg, top_k)
    counts, offsets, perm, _ = orc.permute(ids, lg.shape[1])
    assert np.array_equal(got["topk_ids"].cpu().numpy(), ids)
    assert np.array_equal(got["counts"].cpu().numpy(), counts)
    assert np.array_equal(got["offsets"].cpu().numpy(), offsets)
    assert np.array_equal(got["perm"].cpu().numpy(), perm)
    np.testing.assert_allclose(got["gates"].cpu().numpy(), gates, rtol=1e-6, atol=1e-9)


def test_static_routing_matches_forward_routing_twice_in_a_row(orc):
    cfg = synth.LayerConfig("route_small", 64, 6, 256, 384, 200, routing="zipf", zipf_a=1.2, bit_rule="all16")
    T = cfg.tokens
    first = synth.router_logits(cfg, 0, 0, device="cuda")
    second = synth.router_logits(cfg, 0, 1, device="cuda", tokens=77)        # different size: stale scratch must not leak
    for logits, t in ((first, T), (second, 77)):
        got = B.pw_route_tokens_static(logits.contiguous(), cfg.top_k)
        ref = reference_routing(cfg, logits.contiguous(), t)
        torch.cuda.synchronize()
        for name in ("topk_ids", "counts", "offsets", "perm"):
            assert torch.equal(got[name], ref[name]), name
        assert torch.equal(got["gates"].view(torch.int32), ref["gates"].view(torch.int32))
        check_against_oracle(orc, got, logits, cfg.top_k)
    # and again the first input: same answer as before
    again = B.pw_route_tokens_static(first.contiguous(), cfg.top_k)
    ref = reference_routing(cfg, first.contiguous(), T)
    assert torch.equal(again["perm"], ref["perm"]) and torch.equal(again["counts"], ref["counts"])
    check_against_oracle(orc, again, first, cfg.top_k)


def test_static_routing_rejects_what_does_not_fit():
    big = torch.zeros(70000, 8, device="cuda")
    with pytest.raises(B.PwError) as e:
        B.pw_route_tokens_static(big, 1)            # 70000 pairs > 65536
    assert e.value.status == 6
    wide = torch.zeros(4, 300, device="cuda")
    with pytest.raises(B.PwError) as e:
        B.pw_route_tokens_static(wide, 2)           # more experts than the fixed scratch covers
    assert e.value.status == 6
    with pytest.raises(B.PwError) as e:
        B.pw_route_tokens_static(torch.zeros(4, 8, device="cuda"), 9)
    assert e.value.status == 1
