"""Pins of the observation oracle: routing mass (Eq. 1) and routed-input features (Sec. 3.2).  CPU only.

Checked against a case worked by hand, closed forms (k = E is a plain softmax; identity weights make the
SwiGLU activation elementwise), a literal loop over the (token, choice) pairs, and the properties any weighted
mean / RMS / maximum has.
"""
import math

import numpy as np
import pytest
import scipy.special


@pytest.fixture(scope="module")
def obs(orc):
    from oracle import observe
    return observe


def dense_pages(orc, E, H, F, seed, bits=16, n_shared=0):
    rng = np.random.default_rng(seed)
    pages = []
    for e in range(E + n_shared):
        for u in range(3):
            rows, cols = (H, F) if u == 2 else (F, H)
            w = (rng.standard_normal((rows, cols)) * 0.05).astype(np.float16)
            pages.append(orc.quantize_block(w, 16 if e >= E else bits))
    return pages


def test_worked_example(orc, obs):
    # token 0: logits (ln 3, 0, -10) -> experts 0, 1 with gates 3/4, 1/4; |x_0| = 3
    # token 1: logits (-10, 0, 0)    -> experts 1, 2 with gates 1/2, 1/2; |x_1| = 4
    H = F = 128
    x = np.zeros((2, H), np.float16)
    x[0, 5] = 3.0
    x[1, 7] = -4.0
    logits = np.array([[math.log(3.0), 0.0, -10.0], [-10.0, 0.0, 0.0]], np.float32)
    pages = dense_pages(orc, 3, H, F, seed=1)
    acc = obs.accumulate(x, logits, 2, pages)
    mass, phi = obs.summarize(acc, 3)
    assert np.allclose(mass, [0.375, 0.375, 0.25], rtol=1e-6)
    assert np.allclose(acc[:, 0], [0.75, 0.75, 0.5], rtol=1e-6) and acc[:, 1].tolist() == [1, 2, 1]
    # expert 1 sees token 0 with weight 1/4 and token 1 with weight 1/2
    assert np.allclose(phi[1, 0], [(0.25 * 3 + 0.5 * 4) / 0.75, math.sqrt((0.25 * 9 + 0.5 * 16) / 0.75), 4.0], rtol=1e-6)
    assert np.array_equal(phi[1, 0], phi[1, 1])                  # gate and up blocks share their input
    assert np.allclose(phi[0, 0], [3, 3, 3], rtol=1e-6) and np.allclose(phi[2, 0], [4, 4, 4], rtol=1e-6)


def test_mass_closed_forms(orc, obs):
    rng = np.random.default_rng(2)
    T, E, H, F = 40, 8, 128, 128
    x = rng.standard_normal((T, H)).astype(np.float16)
    logits = rng.standard_normal((T, E)).astype(np.float32)
    pages = dense_pages(orc, E, H, F, seed=3)
    # k = E: every expert is chosen by every token, r is the plain softmax, the denominator is T
    mass, _ = obs.summarize(obs.accumulate(x, logits, E, pages), E)
    assert np.allclose(mass, scipy.special.softmax(logits.astype(np.float64), axis=1).mean(axis=0), rtol=1e-5)
    # k = 1: the gate is 1, mass is the share of tokens
    mass, _ = obs.summarize(obs.accumulate(x, logits, 1, pages), E)
    assert np.allclose(mass, np.bincount(logits.argmax(axis=1), minlength=E) / T, rtol=1e-6)
    for k in (2, 3):
        acc = obs.accumulate(x, logits, k, pages)
        mass, phi = obs.summarize(acc, E)
        assert abs(mass.sum() - 1.0) < 1e-9 and (mass >= 0).all()
        assert abs(acc[:, 0].sum() - T) < 1e-4 and acc[:, 1].sum() == T * k
        live = acc[:, 0] > 0
        assert (phi[live, :, 0] <= phi[live, :, 1] * (1 + 1e-12)).all()       # mean <= RMS <= max
        assert (phi[live, :, 1] <= phi[live, :, 2] * (1 + 1e-12)).all()


def test_literal_pair_loop(orc, obs):
    rng = np.random.default_rng(4)
    T, E, k, H, F = 9, 5, 2, 128, 256
    x = rng.standard_normal((T, H)).astype(np.float16)
    logits = rng.standard_normal((T, E)).astype(np.float32)
    pages = dense_pages(orc, E, H, F, seed=5, bits=4)
    acc = obs.accumulate(x, logits, k, pages)
    ids, gates = orc.router(logits, k)
    dense = [orc.dequantize_block(p).astype(np.float64) for p in pages]
    num = np.zeros(E)
    srn = np.zeros(E)
    srn2 = np.zeros(E)
    mx = np.zeros(E)
    den = 0.0
    for t in range(T):
        for j in range(k):
            e, r = int(ids[t, j]), float(gates[t, j])
            num[e] += r
            den += r
            xt = x[t].astype(np.float64)
            a = dense[3 * e] @ xt
            h = a / (1 + np.exp(-a)) * (dense[3 * e + 1] @ xt)
            n = math.sqrt(float(h @ h))
            srn[e] += r * n
            srn2[e] += r * n * n
            mx[e] = max(mx[e], n)
    mass, phi = obs.summarize(acc, E)
    assert np.allclose(mass, num / den, rtol=1e-12)
    live = num > 0
    assert np.allclose(phi[live, 2, 0], srn[live] / num[live], rtol=1e-10)
    assert np.allclose(phi[live, 2, 1], np.sqrt(srn2[live] / num[live]), rtol=1e-10)
    assert np.allclose(phi[live, 2, 2], mx[live], rtol=1e-10)


def test_identity_weights_make_the_activation_elementwise(orc, obs):
    H = F = 128
    eye = np.eye(H, dtype=np.float16)
    pages = [orc.quantize_block(eye, 16), orc.quantize_block((2 * eye).astype(np.float16), 16),
             orc.quantize_block(eye, 16)]
    rng = np.random.default_rng(6)
    x = rng.standard_normal((7, H)).astype(np.float16)
    acc = obs.accumulate(x, np.zeros((7, 1), np.float32), 1, pages)
    xd = x.astype(np.float64)
    nh = np.sqrt(((2 * xd * xd / (1 + np.exp(-xd))) ** 2).sum(axis=1))       # silu(x) * 2x
    assert np.allclose(acc[0, 5:8], [nh.sum(), (nh ** 2).sum(), nh.max()], rtol=1e-10)
    swapped = np.sqrt(((xd * 2 * xd / (1 + np.exp(-2 * xd))) ** 2).sum(axis=1))   # silu(2x) * x: gate and up exchanged
    assert not np.allclose(nh, swapped, rtol=1e-3)


def test_scaling_accumulation_and_shared_experts(orc, obs):
    rng = np.random.default_rng(7)
    T, E, k, H, F = 12, 4, 2, 128, 128
    x = rng.standard_normal((T, H)).astype(np.float16)
    logits = rng.standard_normal((T, E)).astype(np.float32)
    pages = dense_pages(orc, E, H, F, seed=8, n_shared=1)
    acc = obs.accumulate(x, logits, k, pages, n_shared=1)
    mass, phi = obs.summarize(acc, E)
    # doubling the inputs (exact in fp16) doubles the input norms and leaves the mass alone
    mass2, phi2 = obs.summarize(obs.accumulate((2 * x).astype(np.float16), logits, k, pages, n_shared=1), E)
    assert np.allclose(mass2, mass, rtol=1e-12) and np.allclose(phi2[:, 0], 2 * phi[:, 0], rtol=1e-12)
    # the shared expert takes every token with weight 1 and is not part of the mass
    nx = np.sqrt((x.astype(np.float64) ** 2).sum(axis=1))
    assert acc[E, 0] == T and acc[E, 1] == T and len(mass) == E
    assert np.allclose(phi[E, 0], [nx.mean(), math.sqrt((nx ** 2).mean()), nx.max()], rtol=1e-12)
    # observed tokens accumulate: two calls equal one call on all the tokens
    two = obs.accumulate(x[:5], logits[:5], k, pages, n_shared=1)
    two = obs.accumulate(x[5:], logits[5:], k, pages, n_shared=1, acc=two)
    assert np.allclose(two, acc, rtol=1e-12)
    # an expert without tokens reports zeros
    lg = np.full((3, E), -50.0, np.float32)
    lg[:, 0] = 0.0
    lg[:, 1] = 0.0
    m0, p0 = obs.summarize(obs.accumulate(x[:3], lg, 2, pages, n_shared=1), E)
    assert m0[2] == 0 and m0[3] == 0 and (p0[2] == 0).all() and abs(m0[:2].sum() - 1) < 1e-12
