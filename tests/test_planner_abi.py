"""The library's planner (host code behind the C ABI, no GPU needed) against the planner oracle on random tables:
the same steps in the same order, the same damages, bytes and stage."""
import numpy as np
import pytest

from paper_2607_16184_b200 import binding as B


@pytest.fixture(scope="module")
def pl():
    from oracle import planner
    return planner


def random_tables(rng, L, E, n_shared, with_heads):
    S = E + n_shared
    committed = rng.choice([16, 8, 4], size=(L, S, 3)).astype(np.uint8)
    committed[:, E:] = 16
    supported = rng.random((L, S, 3, 5)) < 0.8
    for lv, b in enumerate((16, 8, 4, 3, 2)):
        supported[..., lv] |= committed == b                 # the committed page exists
    sens = np.sort(rng.random((L, S, 3, 5)).astype(np.float32), axis=-1)
    sens[rng.random((L, S, 3, 5)) < 0.1] = 0.0              # some non-monotone entries: Eq. 4 clamps them
    nbytes = np.broadcast_to(np.array([117440512, 60555264, 31195136, 23855104, 16515072], np.uint64), (L, S, 3, 5)).copy()
    mass = rng.dirichlet(np.ones(E), size=L).astype(np.float32)
    mass[0, :2] = mass[0, 0]                                  # a tie in the ranking
    phi = heads = None
    if with_heads:
        phi = (rng.random((L, S, 3, 3)) * 4).astype(np.float32)
        phi[0, 1] = 0.0                                       # an expert without tokens
        heads = {"w": (rng.standard_normal((3, 5, 5, 3)) * 0.3).astype(np.float32),
                 "a": (rng.standard_normal((3, 5, 5)) * 0.2).astype(np.float32),
                 "c": rng.random((3, 5, 5)).astype(np.float32)}
    return committed, supported, sens, nbytes, mass, phi, heads


@pytest.mark.parametrize("with_heads", [False, True])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_library_planner_matches_the_oracle(pl, seed, with_heads):
    rng = np.random.default_rng(seed)
    L, E, n_shared = 3, 8, 1
    committed, supported, sens, nbytes, mass, phi, heads = random_tables(rng, L, E, n_shared, with_heads)
    shares, mu = np.array([0.25, 0.5, 1.0], np.float32), np.array([4.0, 2.0, 1.0], np.float32)
    floors = np.array([[8, 4, 3], [4, 3, 2], [2, 2, 2]], np.uint8)
    total = int(sum(int(nbytes[l, e, u, (16, 8, 4, 3, 2).index(int(committed[l, e, u]))]) for l in range(L)
                    for e in range(E) for u in range(3)))
    for target in (0, 1, total // 10, total // 3, total // 2, total):
        got, released, stage = B.pw_plan_step(L, E, n_shared, committed, supported, sens, nbytes, mass, shares, mu,
                                              floors, target, phi=phi, heads=heads, alpha=0.7, rho_min=-1.5,
                                              rho_max=1.5, epsilon=1e-6)
        ref, rreleased, rstage = pl.plan(committed.astype(np.int32), supported, sens, nbytes.astype(np.int64), mass,
                                         phi, heads, shares.tolist(), mu.tolist(), floors.astype(np.int32),
                                         float(np.float32(0.7)), -1.5, 1.5, float(np.float32(1e-6)), target, E, n_shared)
        assert [s[:5] for s in got] == [s[:5] for s in ref], target
        assert np.allclose([s[5] for s in got], [s[5] for s in ref], rtol=1e-12, atol=0)
        assert released == rreleased and stage == rstage
        assert released >= target or stage == 2


def test_pressure_bytes_and_argument_errors():
    assert B.pw_kv_pressure_bytes(10, 3, 2 << 20) == 8 * (2 << 20)
    assert B.pw_kv_pressure_bytes(10, 11, 2 << 20) == 0
    ones = np.ones((1, 2, 3, 5))
    with pytest.raises(B.PwError) as e:
        B.pw_plan_step(1, 2, 0, np.full((1, 2, 3), 5, np.uint8), ones, ones, ones, np.ones((1, 2)), [1.0], [1.0], [[2]], 10)
    assert e.value.status == 3                                # a committed bitwidth outside the levels
    with pytest.raises(B.PwError) as e:
        B.pw_plan_step(0, 2, 0, np.full((1, 2, 3), 16, np.uint8), ones, ones, ones, np.ones((1, 2)), [1.0], [1.0], [[2]], 10)
    assert e.value.status == 1


@pytest.mark.parametrize("seed", [0, 3])
def test_library_plan_queue_matches_the_oracle(pl, seed):
    """The plan queue of Alg. 1 behind the C ABI replayed against the oracle's: a run of planner steps with changing
    KV-cache pressure and routing mass; queued candidates, the trigger and the selected plans agree."""
    rng = np.random.default_rng(seed)
    L, E, n_shared = 2, 8, 1
    committed, supported, sens, nbytes, mass, phi, heads = random_tables(rng, L, E, n_shared, True)
    shares, mu = np.array([0.25, 0.5, 1.0], np.float32), np.array([4.0, 2.0, 1.0], np.float32)
    floors = np.array([[8, 4, 3], [4, 3, 2], [2, 2, 2]], np.uint8)
    q = B.PlanQueue(3)
    oq, on = {}, 0
    kv = 64 << 20
    for step, free_blocks in enumerate([40, 12, 3, 30, 0]):                  # threshold 8: pressure at steps 2 and 4
        mass = rng.dirichlet(np.ones(E), size=L).astype(np.float32)          # newer observations every step
        trig, got, released, stage = q.step(L, E, n_shared, committed, supported, sens, nbytes, mass, shares, mu, floors,
                                            8, free_blocks, kv, 5 * kv, phi=phi, heads=heads, alpha=0.7, rho_min=-1.5,
                                            rho_max=1.5, epsilon=1e-6)
        tables = dict(committed=committed.astype(np.int32), supported=supported, sensitivity=sens,
                      page_bytes=nbytes.astype(np.int64), mass=mass, phi=phi, heads=heads, shares=shares.tolist(),
                      mu=mu.tolist(), floors=floors.astype(np.int32), alpha=float(np.float32(0.7)), rho_min=-1.5,
                      rho_max=1.5, eps=float(np.float32(1e-6)), n_experts=E, n_shared=n_shared)
        oq, on, otrig, best = pl.plan_queue_step(oq, on, tables, 8, free_blocks, kv, 5 * kv)
        assert trig == otrig == (free_blocks <= 8)
        for s in range(3):
            target, rel, n, at = q.peek(s)
            assert (target, rel, n, at) == (oq[s][0], oq[s][2], len(oq[s][1]), oq[s][3])
        if trig:
            assert [x[:5] for x in got] == [x[:5] for x in best[0]]
            assert released == best[1] and stage == best[2]
        else:
            assert got == [] and released == 0 and stage == -1
    q.close()
    with pytest.raises(B.PwError):
        B.PlanQueue(0)
