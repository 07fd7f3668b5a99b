"""Pins of the oracle's router, permutation and layer forward (CPU only).

The forward is checked against numpy float64 restatements that use library
matmul / softmax / argsort, against the brute-force all-experts loop, and against
properties that any correct MoE layer has.
"""
import numpy as np
import pytest
import scipy.special


def synth_w(rows, cols, seed):
    rng = np.random.default_rng(seed)
    w = rng.standard_normal((rows, cols)) * 0.02
    w = np.where(rng.random((rows, cols)) < 0.001, w * 10, w)
    return w.astype(np.float16)


def make_layer(orc, E, H, F, bits_of, seed=0, n_shared=0):
    pages, dense = [], []
    for e in range(E + n_shared):
        for u in range(3):
            rows, cols = (H, F) if u == 2 else (F, H)
            w = synth_w(rows, cols, seed * 1000 + e * 3 + u)
            b = 16 if e >= E else bits_of(e, u)
            pg = orc.quantize_block(w, b)
            pages.append(pg)
            dense.append(orc.dequantize_block(pg).astype(np.float64))
    return pages, dense


def np_forward(x16, logits, k, dense, E, n_shared=0):
    """float64 restatement with library routines: softmax, argsort, matmul."""
    x = x16.astype(np.float64)
    T, H = x.shape
    out = np.zeros((T, H))
    order = np.argsort(-logits.astype(np.float64), axis=1, kind="stable")[:, :k]
    for t in range(T):
        sel = order[t]
        g = scipy.special.softmax(logits[t, sel].astype(np.float64))
        for j, e in enumerate(sel):
            Wg, Wu, Wd = dense[3 * e: 3 * e + 3]
            a = Wg @ x[t]
            h = a / (1 + np.exp(-a)) * (Wu @ x[t])
            out[t] += g[j] * (Wd @ h)
        for s in range(n_shared):
            Wg, Wu, Wd = dense[3 * (E + s): 3 * (E + s) + 3]
            a = Wg @ x[t]
            out[t] += Wd @ (a / (1 + np.exp(-a)) * (Wu @ x[t]))
    return out


def test_router_basic_properties(orc):
    rng = np.random.default_rng(0)
    logits = rng.standard_normal((64, 16)).astype(np.float32)
    for k in (1, 2, 6, 16):
        ids, gates = orc.router(logits, k)
        assert np.allclose(gates.sum(axis=1), 1.0, atol=1e-6)
        assert all(len(set(r)) == k for r in ids.tolist())
        ref = np.argsort(-logits, axis=1, kind="stable")[:, :k]
        assert np.array_equal(ids, ref)
        sm = scipy.special.softmax(np.take_along_axis(logits, ref, 1).astype(np.float64), axis=1)
        assert np.allclose(gates, sm, rtol=1e-6, atol=1e-7)
        if k == 1:
            assert (gates == 1.0).all()
        if k == 16:                                    # k = E: plain softmax over all experts
            full = scipy.special.softmax(logits.astype(np.float64), axis=1)
            assert np.allclose(gates, np.take_along_axis(full, ids, 1), rtol=1e-6, atol=1e-7)
        # equals softmax over all E renormalised over the chosen k
        full = scipy.special.softmax(logits.astype(np.float64), axis=1)
        pk = np.take_along_axis(full, ids, 1)
        assert np.allclose(gates, pk / pk.sum(axis=1, keepdims=True), rtol=1e-6, atol=1e-7)


def test_router_ties_and_one_hot(orc):
    logits = np.zeros((3, 8), np.float32)
    ids, gates = orc.router(logits, 3)
    assert ids.tolist() == [[0, 1, 2]] * 3             # equal logits: lowest indices, in index order
    assert np.allclose(gates, 1 / 3)
    logits = np.full((2, 8), -100.0, np.float32)
    logits[0, 5] = 50.0
    logits[1, 2] = 50.0
    logits[1, 7] = 49.0
    ids, gates = orc.router(logits, 2)
    assert ids.tolist() == [[5, 0], [2, 7]]
    assert gates[0, 0] == 1.0 and gates[0, 1] == 0.0
    assert np.isclose(gates[1, 0], 1 / (1 + np.exp(-1.0)), rtol=1e-6)
    # tie exactly at the k-th place
    logits = np.array([[1.0, 3.0, 2.0, 2.0, 2.0, 0.0]], np.float32)
    ids, _ = orc.router(logits, 3)
    assert ids.tolist() == [[1, 2, 3]]
    with pytest.raises(ValueError):
        orc.router(logits, 7)


def test_permutation_is_stable_counting_sort(orc):
    rng = np.random.default_rng(1)
    T, k, E = 97, 3, 11
    ids = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    counts, offsets, perm, inv = orc.permute(ids, E)
    flat = ids.reshape(-1)
    assert np.array_equal(counts, np.bincount(flat, minlength=E))
    assert offsets[0] == 0 and np.array_equal(offsets[1:], np.cumsum(counts))
    assert np.array_equal(perm, np.argsort(flat, kind="stable"))
    assert np.array_equal(np.sort(perm), np.arange(T * k))
    assert np.array_equal(inv[perm], np.arange(T * k))
    for e in range(E):
        seg = perm[offsets[e]: offsets[e + 1]]
        assert (flat[seg] == e).all() and (np.diff(seg) > 0).all()


def test_dense_single_expert_is_plain_swiglu_ffn(orc):
    H, F, T = 128, 256, 5
    pages, dense = make_layer(orc, 1, H, F, lambda e, u: 16, seed=3)
    x = np.random.default_rng(4).standard_normal((T, H)).astype(np.float16)
    logits = np.zeros((T, 1), np.float32)
    out = orc.moe_forward(x, logits, 1, pages)
    xd = x.astype(np.float64)
    a = xd @ dense[0].T
    ref = (a / (1 + np.exp(-a)) * (xd @ dense[1].T)) @ dense[2].T
    assert np.allclose(out, ref, rtol=2e-6, atol=1e-7)
    # a transposed operand or swapped gate/up would not survive this
    wrong = ((xd @ dense[1].T) / (1 + np.exp(-(xd @ dense[1].T))) * a) @ dense[2].T
    assert not np.allclose(out, wrong, rtol=1e-3, atol=1e-5)


@pytest.mark.parametrize("n_shared", [0, 2])
def test_mixed_bit_layer_against_numpy_and_brute_force(orc, n_shared):
    E, k, H, F, T = 8, 2, 256, 512, 16
    bits = [16, 8, 4, 3, 2]
    pages, dense = make_layer(orc, E, H, F, lambda e, u: bits[(e * 3 + u) % 5], seed=7, n_shared=n_shared)
    rng = np.random.default_rng(8)
    x = rng.standard_normal((T, H)).astype(np.float16)
    logits = rng.standard_normal((T, E)).astype(np.float32)
    out = orc.moe_forward(x, logits, k, pages, n_shared=n_shared)
    ref = np_forward(x, logits, k, dense, E, n_shared)
    scale = np.abs(ref).max()
    assert np.abs(out - ref).max() <= 2e-6 * scale
    bf = orc.moe_forward(x, logits, k, pages, n_shared=n_shared, brute_force=True)
    assert np.abs(out - bf).max() <= 1e-6 * scale
    # token subset computes the same rows and leaves the rest untouched
    sub = orc.moe_forward(x, logits, k, pages, n_shared=n_shared, tokens=[3, 9])
    assert np.array_equal(sub[[3, 9]], out[[3, 9]]) and np.isnan(sub[0]).all()


def test_token_permutation_equivariance_and_uniform_table(orc):
    E, k, H, F, T = 4, 2, 128, 256, 12
    pages, dense = make_layer(orc, E, H, F, lambda e, u: 4, seed=5)      # uniform-bitwidth table
    rng = np.random.default_rng(6)
    x = rng.standard_normal((T, H)).astype(np.float16)
    logits = rng.standard_normal((T, E)).astype(np.float32)
    out = orc.moe_forward(x, logits, k, pages)
    p = rng.permutation(T)
    out_p = orc.moe_forward(x[p], logits[p], k, pages)
    assert np.array_equal(out_p, out[p])
    ref = np_forward(x, logits, k, dense, E)
    assert np.abs(out - ref).max() <= 2e-6 * np.abs(ref).max()


def test_output_depends_only_on_committed_pages(orc):
    # lowering one block changes exactly the tokens routed to that expert
    E, k, H, F, T = 4, 1, 128, 256, 10
    pages, _ = make_layer(orc, E, H, F, lambda e, u: 8, seed=12)
    rng = np.random.default_rng(13)
    x = rng.standard_normal((T, H)).astype(np.float16)
    logits = rng.standard_normal((T, E)).astype(np.float32)
    out = orc.moe_forward(x, logits, k, pages)
    ids, _ = orc.router(logits, k)
    pages2 = list(pages)
    pages2[3 * 2 + 2] = orc.demote_block(pages[3 * 2 + 2], 2)           # expert 2, down block, 8 -> 2
    out2 = orc.moe_forward(x, logits, k, pages2)
    hit = ids[:, 0] == 2
    assert hit.any() and (~hit).any()
    assert np.array_equal(out[~hit], out2[~hit])
    assert (np.abs(out[hit] - out2[hit]).max(axis=1) > 0).all()
