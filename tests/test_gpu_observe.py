"""GPU parity of the observation taps (routing mass, Eq. 1; routed-input features, Sec. 3.2) against the
numpy oracle.  Tolerances: the token-norm sums differ from float64 only by fp32 summation order (5e-5); the
activation-norm sums also carry the fp16 rounding of the SwiGLU rows the forward call stores (2e-3); pair
counts are exact."""
import numpy as np
import pytest
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth

from util_gpu import build_layer, export_to_oracle, make_ctx

pytestmark = pytest.mark.gpu

RTOL_X, RTOL_H = 5e-5, 2e-3


@pytest.fixture(scope="module")
def obs(orc):
    from oracle import observe
    return observe


def compare(acc_gpu, acc_ref):
    live = ~np.isnan(acc_ref[:, 5])
    assert np.array_equal(acc_gpu[:, 1], acc_ref[:, 1])
    assert np.allclose(acc_gpu[:, [0, 2, 3, 4]], acc_ref[:, [0, 2, 3, 4]], rtol=RTOL_X, atol=1e-7)
    assert np.allclose(acc_gpu[live][:, 5:8], acc_ref[live][:, 5:8], rtol=RTOL_H, atol=1e-7)


def run_case(orc, obs, cfg, mode, token_counts, bits=None, experts=None):
    T_max = max(token_counts)
    ctx = make_ctx(cfg, max_tokens=T_max, n_layers=1)
    try:
        pages, _ = build_layer(ctx, cfg, 0, bits)
        opages = [export_to_oracle(ctx, p, orc) for p in pages]
        acc_dev = ctx.pw_observe(True)
        ref = None
        for i, T in enumerate(token_counts):
            x = synth.activations(cfg, device="cuda", tokens=T_max)[i:i + T].contiguous()
            lg = synth.router_logits(cfg, device="cuda", tokens=T_max)[i:i + T].contiguous()
            ctx.pw_moe_forward(0, x, lg, cfg.top_k, mode=mode)
            if callable(experts):
                experts = experts(lg.cpu().numpy())
            ref = obs.accumulate(x.cpu().numpy(), lg.cpu().numpy(), cfg.top_k, opages, n_shared=cfg.n_shared,
                                 acc=ref, experts=experts)
        mass, phi = ctx.pw_observation_summary(0)
        torch.cuda.synchronize()
        assert ctx.pw_last_device_status() == 0
        got = acc_dev[0].cpu().numpy().astype(np.float64)
        compare(got, ref)
        live = ~np.isnan(ref[:, 5])
        rmass, rphi = obs.summarize(np.nan_to_num(ref), cfg.n_experts)
        assert np.allclose(mass.cpu().numpy(), rmass, rtol=RTOL_X, atol=1e-8)
        gphi = phi.cpu().numpy()
        assert np.allclose(gphi[:, :2], rphi[:, :2], rtol=RTOL_X, atol=1e-7)
        assert np.allclose(gphi[live, 2], rphi[live, 2], rtol=RTOL_H, atol=1e-7)
        return got
    finally:
        ctx.close()


@pytest.mark.parametrize("mode", [B.PW_MODE_SIMT, B.PW_MODE_TENSOR])
def test_tiny_layer_two_calls_accumulate(orc, obs, mode):
    run_case(orc, obs, synth.CONFIGS["tiny_cover"], mode, [16, 9])


@pytest.mark.parametrize("T", [1, 3, 33, 130])
def test_ragged_token_counts(orc, obs, T):
    run_case(orc, obs, synth.CONFIGS["tiny"], B.PW_MODE_TENSOR, [T])


def test_shared_experts_and_experts_without_tokens(orc, obs):
    cfg = synth.LayerConfig("fg_small", 64, 6, 256, 384, 40, n_shared=2, routing="zipf", zipf_a=1.2,
                            bit_rule="int4_10fp16_20int2")
    got = run_case(orc, obs, cfg, B.PW_MODE_TENSOR, [40])
    assert (got[:64, 1] == 0).any()                  # Zipf routing of 40 tokens leaves some experts idle
    assert (got[64:, 0] == 40).all()                 # a shared expert takes every token with weight 1


def test_taps_are_reproducible_resettable_and_optional(orc, obs):
    cfg = synth.CONFIGS["tiny"]
    ctx = make_ctx(cfg, n_layers=1)
    try:
        pages, _ = build_layer(ctx, cfg, 0)
        x = synth.activations(cfg, device="cuda")
        lg = synth.router_logits(cfg, device="cuda")
        with pytest.raises(B.PwError) as ei:
            ctx.pw_observation_summary(0)
        assert ei.value.status == 5                # PW_ERR_STATE: the taps are off
        n0 = ctx.pw_launch_count()
        out_off = ctx.pw_moe_forward(0, x, lg, cfg.top_k).clone()
        per_call_off = ctx.pw_launch_count() - n0
        a = ctx.pw_observe(True)
        n0 = ctx.pw_launch_count()
        out_on = ctx.pw_moe_forward(0, x, lg, cfg.top_k).clone()
        assert ctx.pw_launch_count() - n0 == per_call_off + 1
        first = a.clone()
        b = ctx.pw_observe(True)                      # fresh accumulators
        ctx.pw_moe_forward(0, x, lg, cfg.top_k)
        torch.cuda.synchronize()
        assert torch.equal(out_off, out_on)           # the taps never touch the layer's result
        assert torch.equal(first, b)                  # same call, same bits
        ctx.pw_moe_forward(0, x, lg, cfg.top_k)
        torch.cuda.synchronize()
        assert torch.equal(b[0, :, 1], 2 * first[0, :, 1])
        ctx.pw_observe(False)
        snapshot = b.clone()
        ctx.pw_moe_forward(0, x, lg, cfg.top_k)
        torch.cuda.synchronize()
        assert torch.equal(b, snapshot)
        assert ctx.pw_last_device_status() == 0
    finally:
        ctx.close()


def test_mixtral_decode_full_size(orc, obs):
    # every expert's mass and token-norm sums; the activation-norm sums of two experts (their weights are
    # dequantized by the oracle, 117 M values each)
    cfg = synth.CONFIGS["mixtral_decode"]

    def pick(lg):                                    # the busiest expert and the least busy one that has tokens
        ids, _ = orc.router(lg, cfg.top_k)
        busy = np.bincount(ids.reshape(-1), minlength=cfg.n_experts)
        return [int(np.argmax(busy)), int(np.argmax(np.where(busy > 0, -busy, -10 ** 9)))]

    run_case(orc, obs, cfg, B.PW_MODE_AUTO, [cfg.tokens], experts=pick)
