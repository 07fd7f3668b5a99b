"""Pins of the planner oracle (Sec. 3.2, Alg. 1, Eqs. 4-8): the equations on hand-computed values, the
selection on a case worked by hand, and the properties the text states (floors, protection of hot experts,
stage relaxation, largest safe reduction, prefix property in the target).  CPU only."""
import math

import numpy as np
import pytest


@pytest.fixture(scope="module")
def pl():
    from oracle import planner
    return planner


def test_equations_on_hand_values(pl):
    # Eq. 7: threshold 10 free blocks, 3 free, 2 MiB per block -> (10 + 1 - 3) blocks
    assert pl.target_bytes(10, 3, 2 << 20) == 8 * (2 << 20)
    assert pl.target_bytes(10, 11, 2 << 20) == 0 and pl.target_bytes(10, 50, 1) == 0
    # Eq. 4: only an increase of the sensitivity counts
    assert pl.global_damage(1.5, 4.0) == 2.5 and pl.global_damage(4.0, 1.5) == 0.0
    # Eqs. 5-6: rho = 1*2 + 0*5 + 0*7 - 1 = 1; eta = exp(2 * 0.5 * 1) = e; clipped at 0.5 -> exp(0.5)
    assert math.isclose(pl.prompt_factor((2, 5, 7), (1, 0, 0), -1.0, 0.5, 2.0, -3.0, 3.0), math.e, rel_tol=1e-12)
    assert math.isclose(pl.prompt_factor((2, 5, 7), (1, 0, 0), -1.0, 0.5, 2.0, -3.0, 0.5), math.exp(0.5), rel_tol=1e-12)
    assert math.isclose(pl.prompt_factor((0, 0, 0), (1, 1, 1), -9.0, 1.0, 1.0, -2.0, 2.0), math.exp(-2.0), rel_tol=1e-12)
    # Eq. 8: the floor
    assert pl.predicted_damage(3.0, 2.0, 0.5, 1e-6) == 3.0 and pl.predicted_damage(3.0, 0.0, 0.5, 1e-6) == 1e-6


def tiny_instance(n_experts=2):
    L, S = 1, n_experts
    committed = np.full((L, S, 3), 16, np.int32)
    supported = np.zeros((L, S, 3, 5), bool)
    supported[..., 0] = True                       # every block exists at 16 bits
    supported[:, :, 0, 2] = True                   # the gate blocks also at 4 and 2 bits
    supported[:, :, 0, 4] = True
    sens = np.zeros((L, S, 3, 5))
    nbytes = np.zeros((L, S, 3, 5), np.int64)
    nbytes[..., 0], nbytes[..., 2], nbytes[..., 4] = 100, 30, 20
    return committed, supported, sens, nbytes


def run(pl, committed, supported, sens, nbytes, target, mass=None, shares=(1.0,), mu=(1.0,), floors=((2,),), **kw):
    L, S, _ = committed.shape
    mass = np.full((L, S), 1.0 / S) if mass is None else mass
    return pl.plan(committed, supported, sens, nbytes, mass, kw.get("phi"), kw.get("heads"), shares, mu,
                   np.asarray(floors), kw.get("alpha", 1.0), -5.0, 5.0, 1e-9, target, S, 0)


def test_selection_worked_by_hand(pl):
    committed, supported, sens, nbytes = tiny_instance()
    # block A = (expert 0, gate): 16->4 costs 7 for 70 bytes (0.1 per byte), 4->2 costs 2 for 10 bytes (0.2)
    sens[0, 0, 0, 2], sens[0, 0, 0, 4] = 7.0, 9.0
    # block B = (expert 1, gate): 16->4 costs 14 for 70 bytes (0.2), 4->2 costs 0.5 for 10 bytes (0.05)
    sens[0, 1, 0, 2], sens[0, 1, 0, 4] = 14.0, 14.5
    steps, released, stage = run(pl, committed, supported, sens, nbytes, 150)
    # A 16->4 first; then a tie at 0.2 which the lower block wins (A 4->2); then B 16->4 reaches 150 bytes
    assert [(s[1], s[3], s[4]) for s in steps] == [(0, 16, 4), (0, 4, 2), (1, 16, 4)]
    assert released == 150 and stage == 0 and [s[5] for s in steps] == [7.0, 2.0, 14.0]
    steps, released, _ = run(pl, committed, supported, sens, nbytes, 151)     # one byte more: B's cheap second step
    assert [(s[1], s[3], s[4]) for s in steps][-1] == (1, 4, 2) and released == 160
    assert run(pl, committed, supported, sens, nbytes, 0)[0] == []


def test_buckets_floors_and_stages(pl):
    committed, supported, sens, nbytes = tiny_instance()
    sens[:, :, 0, 2], sens[:, :, 0, 4] = 1.0, 2.0          # both experts equally sensitive
    mass = np.array([[0.9, 0.1]])                            # expert 0 is hot
    assert pl.buckets_of_layer(mass[0], (0.5, 1.0)).tolist() == [0, 1]
    assert pl.buckets_of_layer(np.array([0.2, 0.2, 0.6, 0.0]), (0.25, 0.5, 1.0)).tolist() == [1, 2, 0, 2]
    kw = dict(mass=mass, shares=(0.5, 1.0), mu=(10.0, 1.0))
    # stage 0 keeps the hot bucket at 16 bits: only expert 1 moves, and 80 bytes are all it can give
    steps, released, stage = run(pl, committed, supported, sens, nbytes, 80, floors=((16, 2), (4, 2)), **kw)
    assert stage == 0 and released == 80 and {s[1] for s in steps} == {1}
    # 100 bytes need the relaxed floors of stage 1; the hot expert's step is 10 times as expensive, so it comes
    # after both steps of the cold one and stops at its floor of 4 bits
    steps, released, stage = run(pl, committed, supported, sens, nbytes, 100, floors=((16, 2), (4, 2)), **kw)
    assert stage == 1 and [(s[1], s[3], s[4]) for s in steps] == [(1, 16, 4), (1, 4, 2), (0, 16, 4)] and released == 150
    assert steps[2][5] == 10.0
    # nothing satisfies 1000 bytes: the largest safe reduction of the last stage comes back
    steps, released, stage = run(pl, committed, supported, sens, nbytes, 1000, floors=((16, 2), (4, 2)), **kw)
    assert stage == 1 and released == 150 and len(steps) == 3


def test_prompt_factor_reorders_and_idle_experts_keep_the_prior(pl):
    committed, supported, sens, nbytes = tiny_instance()
    sens[:, :, 0, 2] = 1.0
    heads = {"w": np.zeros((3, 5, 5, 3)), "a": np.zeros((3, 5, 5)), "c": np.ones((3, 5, 5))}
    heads["w"][0, 0, 2] = (1.0, 0.0, 0.0)                  # gate blocks, 16 -> 4: rho = mean input norm
    phi = np.zeros((1, 2, 3, 3))
    phi[0, 0, 0] = (2.0, 2.0, 2.0)                           # expert 0 sees large inputs: eta = e^2, expert 1 none
    steps, _, _ = run(pl, committed, supported, sens, nbytes, 70, phi=phi, heads=heads)
    assert [(s[1], s[5]) for s in steps] == [(1, 1.0)]       # the idle expert keeps eta = 1 and goes first
    phi[0, 1, 0] = (3.0, 3.0, 3.0)
    steps, _, _ = run(pl, committed, supported, sens, nbytes, 70, phi=phi, heads=heads)
    assert steps[0][1] == 0 and math.isclose(steps[0][5], math.exp(2.0), rel_tol=1e-12)


def test_properties_on_random_tables(pl):
    rng = np.random.default_rng(5)
    L, E, n_shared = 2, 6, 1
    S = E + n_shared
    committed = rng.choice([16, 8], size=(L, S, 3)).astype(np.int32)
    committed[:, E:] = 16
    supported = np.ones((L, S, 3, 5), bool)
    supported[..., 3] = rng.random((L, S, 3)) < 0.5         # 3 bits only for some blocks
    sens = np.sort(rng.random((L, S, 3, 5)), axis=-1)        # lower bitwidth, higher sensitivity
    nbytes = np.broadcast_to(np.array([1000, 520, 270, 210, 150], np.int64), (L, S, 3, 5)).copy()
    mass = rng.dirichlet(np.ones(E), size=L)
    floors = np.array([[8, 4, 2], [4, 3, 2]])
    args = (committed, supported, sens, nbytes, mass, None, None, (0.2, 0.6, 1.0), (4.0, 2.0, 1.0), floors, 1.0,
            -1.0, 1.0, 1e-9)
    full, released_all, _ = pl.plan(*args, 10 ** 9, E, n_shared)
    assert all(s[1] < E for s in full)                       # shared experts are never touched
    bucket = np.stack([pl.buckets_of_layer(mass[l], (0.2, 0.6, 1.0)) for l in range(L)])
    cur = committed.copy()
    for (l, e, u, b, b2, d) in full:
        assert cur[l, e, u] == b and b2 < b and b2 >= floors[1, bucket[l, e]] and d >= 1e-9
        lv = [x for i, x in enumerate(pl.LEVELS) if supported[l, e, u, i] and x < b]
        assert b2 == max(lv)                                 # the next lower supported bitwidth, never a jump
        cur[l, e, u] = b2
    assert released_all == sum(nbytes[l, e, u, pl.LEVELS.index(b)] - nbytes[l, e, u, pl.LEVELS.index(b2)]
                               for (l, e, u, b, b2, d) in full)
    # within a stage a smaller target gives a prefix of the larger target's plan
    small, released, stage = pl.plan(*args, 900, E, n_shared)
    assert released >= 900 and stage == 0
    bigger, _, stage2 = pl.plan(*args, 2500, E, n_shared)
    if stage2 == 0:
        assert bigger[: len(small)] == small


def test_plan_queue_step_refreshes_and_selects(pl):
    """Alg. 1: without pressure the queue is refreshed and no plan leaves it; under pressure the selected plan is
    the one a fresh planner step returns for the target of Eq. 7; a later step replaces older candidates."""
    L, E = 1, 4
    committed = np.full((L, E, 3), 16, np.int32)
    supported = np.ones((L, E, 3, 5), bool)
    sens = np.tile(np.array([0.0, 1.0, 2.0, 4.0, 8.0], np.float32), (L, E, 3, 1))
    sens[0, 0] *= 0.1                                           # expert 0 is the cheapest to lower
    nbytes = np.tile(np.array([1000, 600, 400, 300, 200], np.int64), (L, E, 3, 1))
    mass = np.array([[0.1, 0.2, 0.3, 0.4]], np.float32)
    tables = dict(committed=committed, supported=supported, sensitivity=sens, page_bytes=nbytes, mass=mass, phi=None,
                  heads=None, shares=[0.5, 1.0], mu=[2.0, 1.0], floors=np.array([[8, 4], [4, 2]], np.int32), alpha=1.0,
                  rho_min=-1.0, rho_max=1.0, eps=1e-9, n_experts=E, n_shared=0)
    q, n, trig, best = pl.plan_queue_step({}, 0, tables, free_block_threshold=4, free_blocks=9, kv_block_bytes=500,
                                          lookahead_bytes=900)
    assert not trig and best is None and n == 1
    assert q[0][0] == 900 and q[0][3] == 1 and q[0][2] >= 900   # candidates built for the look-ahead bytes
    # pressure: 4 + 1 - 1 = 4 blocks of 500 bytes
    q, n, trig, best = pl.plan_queue_step(q, n, tables, 4, 1, 500, 900)
    assert trig and n == 2 and q[0][0] == 2000 and q[1][3] == 2
    fresh = pl.plan(target=2000, **tables)
    assert best[0] == fresh[0] and best[1] == fresh[1] and best[2] == fresh[2]
    # a target the first stage cannot meet (its floors allow 12 blocks x 400 + ... ): falls to the later stage
    big = sum(1000 - 400 for _ in range(6)) + sum(1000 - 600 for _ in range(6)) + 1
    q, n, trig, best = pl.plan_queue_step(q, n, tables, big // 500 + 1, 0, 500, 0)
    assert trig and best[2] == 1 and best[1] >= pl.target_bytes(big // 500 + 1, 0, 500)
