"""Oracle of the runtime planner's scoring and selection (Sec. 3.2, Alg. 1, Eqs. 4-8).  TEST INFRASTRUCTURE ONLY.

Plain Python / numpy in float64, one function per equation, then the selection as the text states it:
"each legal bitwidth reduction is one step; steps are sorted by predicted damage per released byte and the
cheapest are taken until the target is met; caps are relaxed only when the current caps cannot provide enough
bytes; if no legal plan satisfies the target, the largest safe reduction is returned".

Readings (the paper leaves these open; the calibrated constants are the caller's):
  - a step lowers one linear-block from its current bitwidth to the next lower bitwidth it supports; a block's
    further steps become available once the one before has been taken, so "sorted and taken greedily" means:
    repeatedly take the available step with the smallest damage per byte (ties: lower block index);
  - routing buckets: the experts of a layer are ranked by routing mass, hottest first (ties: lower expert
    index), and bucket j holds the ranks below share[j] * E (shares ascending, the last one 1); shared
    experts are never touched;
  - stages: stage s has its own bitwidth floor per bucket; the stages are tried in order and the plan of the
    first stage that reaches the target is returned, otherwise that of the last stage;
  - the prompt factor eta is 1 for a block whose expert saw no token (phi = 0 would otherwise feed the head
    an input it was not fitted on), and 1 everywhere when no heads are given;
  - the plan queue and the pressure trigger of Alg. 1 are the caller's loop: this is one scoring + selection.
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np

LEVELS = (16, 8, 4, 3, 2)


def target_bytes(free_block_threshold: int, free_blocks: int, kv_block_bytes: int) -> int:
    """Eq. 7: D = max(0, T_blk + 1 - F_blk) * B_KV."""
    return max(0, free_block_threshold + 1 - free_blocks) * kv_block_bytes


def global_damage(s_from: float, s_to: float) -> float:
    """Eq. 4: g = max(s^{b'} - s^{b}, 0) for b' < b."""
    return max(s_to - s_from, 0.0)


def prompt_factor(phi: Sequence[float], w: Sequence[float], a: float, c: float, alpha: float, rho_min: float,
                  rho_max: float) -> float:
    """Eqs. 5-6: eta = exp(alpha * c * clip(w . phi + a, rho_min, rho_max))."""
    rho = float(np.dot(np.asarray(w, np.float64), np.asarray(phi, np.float64)) + a)
    return math.exp(alpha * c * min(max(rho, rho_min), rho_max))


def predicted_damage(mu: float, g: float, eta: float, eps: float) -> float:
    """Eq. 8: d = max(eps, mu * g * eta)."""
    return max(eps, mu * g * eta)


def buckets_of_layer(mass: np.ndarray, shares: Sequence[float]) -> np.ndarray:
    """Bucket index of every routed expert of one layer (0 = hottest)."""
    E = len(mass)
    order = sorted(range(E), key=lambda e: (-float(mass[e]), e))
    out = np.zeros(E, np.int32)
    for rank, e in enumerate(order):
        j = 0
        while j < len(shares) - 1 and rank >= shares[j] * E:
            j += 1
        out[e] = j
    return out


def plan(committed: np.ndarray, supported: np.ndarray, sensitivity: np.ndarray, page_bytes: np.ndarray,
         mass: np.ndarray, phi: Optional[np.ndarray], heads: Optional[dict], shares: Sequence[float],
         mu: Sequence[float], floors: np.ndarray, alpha: float, rho_min: float, rho_max: float, eps: float,
         target: int, n_experts: int, n_shared: int) -> Tuple[List[Tuple[int, int, int, int, int, float]], int, int]:
    """One planner step.

    committed [L, S, 3] bitwidths q_i; supported [L, S, 3, 5] bool per level of LEVELS; sensitivity and
    page_bytes [L, S, 3, 5]; mass [L, E]; phi [L, S, 3, 3] or None; heads {"w": [3, 5, 5, 3], "a": [3, 5, 5],
    "c": [3, 5, 5]} indexed (kind, from level, to level) or None; floors [n_stages, n_buckets] bitwidths.
    Returns (steps, released bytes, stage used); a step is (layer, expert, kind, from bits, to bits, damage).
    """
    L, S, _ = committed.shape
    E = n_experts
    result = None
    for stage in range(floors.shape[0]):
        cur = committed.copy()
        released = 0
        steps = []
        bucket = np.stack([buckets_of_layer(mass[l], shares) for l in range(L)])

        def next_step(l, e, u):
            """(ratio, damage, bytes, to_bits) of the block's next legal step, or None."""
            b = int(cur[l, e, u])
            li = LEVELS.index(b)
            for lj in range(li + 1, len(LEVELS)):
                if supported[l, e, u, lj]:
                    b2 = LEVELS[lj]
                    if b2 < int(floors[stage, bucket[l, e]]):
                        return None
                    g = global_damage(float(sensitivity[l, e, u, li]), float(sensitivity[l, e, u, lj]))
                    eta = 1.0
                    if heads is not None and phi is not None and np.any(phi[l, e, u] != 0):
                        eta = prompt_factor(phi[l, e, u], heads["w"][u, li, lj], float(heads["a"][u, li, lj]),
                                            float(heads["c"][u, li, lj]), alpha, rho_min, rho_max)
                    d = predicted_damage(float(mu[bucket[l, e]]), g, eta, eps)
                    delta = int(page_bytes[l, e, u, li]) - int(page_bytes[l, e, u, lj])
                    return d / delta, d, delta, b2
            return None

        while released < target:
            best = None
            for l in range(L):
                for e in range(E):                      # shared experts (e >= E) are never touched
                    for u in range(3):
                        ns = next_step(l, e, u)
                        if ns is not None and (best is None or ns[0] < best[0][0]):
                            best = (ns, l, e, u)
            if best is None:
                break
            (ratio, d, delta, b2), l, e, u = best
            steps.append((l, e, u, int(cur[l, e, u]), b2, d))
            cur[l, e, u] = b2
            released += delta
        result = (steps, released, stage)
        if released >= target:
            break
    return result


def plan_queue_step(queue: dict, steps_taken: int, tables: dict, free_block_threshold: int, free_blocks: int,
                    kv_block_bytes: int, lookahead_bytes: int):
    """One PlanStep of Alg. 1 with its plan queue.  ``queue`` maps stage -> (target, steps, released bytes,
    refreshed at); ``tables`` are the keyword arguments of plan() without ``target``.  The byte target is Eq. 7;
    every stage's candidate plan is rebuilt for it (for ``lookahead_bytes`` while there is no pressure) and replaces
    the stage's entry; under pressure the candidate of the first stage that meets the target is returned, else the
    last stage's.  Returns (queue, steps taken, triggered, plan or None)."""
    D = target_bytes(free_block_threshold, free_blocks, kv_block_bytes)
    triggered = D > 0
    target = D if triggered else lookahead_bytes
    floors = tables["floors"]
    queue = dict(queue)
    steps_taken += 1
    for s in range(floors.shape[0]):
        one = dict(tables, floors=floors[s:s + 1])                  # GreedySelect under the floors of stage s alone
        st, released, _ = plan(target=target, **one)
        queue[s] = (target, st, released, steps_taken)
    best = None
    if triggered:
        best = floors.shape[0] - 1
        for s in range(floors.shape[0]):
            if queue[s][2] >= D:
                best = s
                break
        best = (queue[best][1], queue[best][2], best)
    return queue, steps_taken, triggered, best
