"""The seeded input generator: shapes, determinism and the stated distributions (CPU only)."""
import numpy as np
import torch

from paper_2607_16184_b200 import synth


def test_block_weights_distribution_and_determinism():
    cfg = synth.CONFIGS["tiny"]
    a = synth.block_weights(cfg, 0, 1, 0)
    b = synth.block_weights(cfg, 0, 1, 0)
    c = synth.block_weights(cfg, 0, 1, 1)
    assert a.dtype == torch.float16 and tuple(a.shape) == (512, 256)
    assert torch.equal(a, b) and not torch.equal(a, c)
    assert tuple(synth.block_weights(cfg, 0, 0, 2).shape) == (256, 512)
    big = torch.cat([synth.block_weights(cfg, 0, e, 0).float().flatten() for e in range(8)])
    assert abs(big.std().item() - 0.02 * (1 + 0.001 * 99) ** 0.5) < 2e-3
    assert 0.0002 < (big.abs() > 0.1).float().mean().item() < 0.002      # the x10 outliers


def test_bit_assignments():
    b = synth.assign_bits(synth.CONFIGS["mixtral_decode"])
    assert b.shape == (8, 3)
    assert sorted(np.bincount(b.reshape(-1), minlength=17)[[16, 8, 4, 3, 2]].tolist()) == [2, 3, 6, 6, 7]
    assert np.bincount(b.reshape(-1), minlength=17)[4] == 7
    b = synth.assign_bits(synth.CONFIGS["finegrained_decode"])
    assert b.shape == (66, 3) and (b[64:] == 16).all()
    cnt = np.bincount(b[:64].reshape(-1), minlength=17)
    assert cnt[16] == 19 and cnt[2] == 38 and cnt[4] == 135
    b = synth.assign_bits(synth.CONFIGS["tiny_cover"])
    assert {(int(b[e, u]), u) for e in range(8) for u in range(3)} == {(q, u) for q in synth.BITS for u in range(3)}
    assert set(np.unique(synth.assign_bits(synth.CONFIGS["mixtral_prefill"]))) <= {16, 8, 4}
    assert (synth.assign_bits(synth.CONFIGS["demote_under_load"], 5) == 16).all()
    assert np.array_equal(synth.assign_bits(synth.CONFIGS["tiny"]), synth.assign_bits(synth.CONFIGS["tiny"]))


def test_zipf_logits_follow_the_stated_popularity():
    cfg = synth.CONFIGS["mixtral_decode"]
    l = synth.router_logits(cfg, tokens=20000)
    assert l.dtype == torch.float32 and tuple(l.shape) == (20000, 8)
    freq = np.bincount(l.argmax(dim=1).numpy(), minlength=8) / 20000
    assert np.abs(freq - synth.zipf_reference_probs(cfg)).max() < 0.015   # Gumbel-max: top-1 frequencies are Zipf


def test_demote_schedule():
    cfg = synth.CONFIGS["demote_under_load"]
    s = synth.demote_schedule(cfg)
    assert len(s) == 256 and len(set(s)) == 256
    assert all(0 <= l < 32 and 0 <= e < 8 and 0 <= u < 3 for l, e, u in s)
