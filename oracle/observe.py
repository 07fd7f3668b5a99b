"""Oracle of the observation taps: routing mass and routed-input features.  TEST INFRASTRUCTURE ONLY.

Plain numpy in float64, written from the definitions:

* routing mass of expert e of a layer (Eq. 1): the routing weight that went to e, summed over the
  observed tokens t and their top-k choices, divided by the routing weight of all experts;
* the routed-input feature vector phi_i of a linear-block i (Sec. 3.2, prompt residuals): routing-weighted
  mean input norm, routing-weighted RMS input norm and maximum input norm over the tokens routed to the
  block's expert.

Readings (the paper gives no formula for phi):
  - the routing weight r_{t,k} is the gate the layer multiplies the expert's output with (softmax over the k
    selected logits); a shared expert takes every token with weight 1 and has no routing mass;
  - "input norm" is the Euclidean norm of the vector the block multiplies: the token's hidden state x_t for a
    gate or up block, the SwiGLU activation silu(W_gate x_t) * (W_up x_t) of that expert for its down block;
  - weighted mean = sum r n / sum r, weighted RMS = sqrt(sum r n^2 / sum r), maximum = max n, over the pairs
    (t, k) routed to the expert; an expert nobody was routed to has phi = 0;
  - "observed tokens" accumulate over calls: the sums run over every call since the last reset.

Only tests, the smoke check and the benchmark's CPU legs import this module.  Routing comes from the
oracle's router; nothing here is shared with the CUDA sources.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np

from . import oracle as orc

FIELDS = ("sum_r", "pairs", "sum_r_nx", "sum_r_nx2", "max_nx", "sum_r_nh", "sum_r_nh2", "max_nh")


def swiglu_rows(x: np.ndarray, gate: orc.Page, up: orc.Page) -> np.ndarray:
    """silu(W_gate x) * (W_up x) for the rows of x ([n, H] float64), weights as their pages decode."""
    wg = orc.dequantize_block(gate).astype(np.float64)
    wu = orc.dequantize_block(up).astype(np.float64)
    g = x @ wg.T
    u = x @ wu.T
    return g / (1.0 + np.exp(-g)) * u


def accumulate(hidden_fp16: np.ndarray, logits: np.ndarray, k: int, pages: Sequence[orc.Page], n_shared: int = 0,
               acc: Optional[np.ndarray] = None, experts: Optional[Sequence[int]] = None) -> np.ndarray:
    """Adds one layer call to the accumulators ([S, 8] float64, columns as FIELDS) and returns them.

    ``experts`` restricts the activation-norm columns (which need the expert's weights) to those segments;
    the other segments get NaN there.  Everything else is always computed.
    """
    x = np.asarray(hidden_fp16, np.float16).astype(np.float64)
    T = x.shape[0]
    E = logits.shape[1]
    S = E + n_shared
    if acc is None:
        acc = np.zeros((S, len(FIELDS)), np.float64)
    ids, gates = orc.router(logits, k)
    nx = np.sqrt((x * x).sum(axis=1))
    for s in range(S):
        if s < E:
            tt, kk = np.nonzero(ids == s)           # the pairs (t, k) with z_{t,k} = s
            r = gates[tt, kk].astype(np.float64)
        else:
            tt = np.arange(T)
            r = np.ones(T, np.float64)
        if tt.size == 0:
            continue
        a = acc[s]
        a[0] += r.sum()
        a[1] += tt.size
        a[2] += (r * nx[tt]).sum()
        a[3] += (r * nx[tt] ** 2).sum()
        a[4] = max(a[4], nx[tt].max())
        if experts is not None and s not in experts:
            a[5:8] = np.nan
            continue
        h = swiglu_rows(x[tt], pages[s * 3 + 0], pages[s * 3 + 1])
        nh = np.sqrt((h * h).sum(axis=1))
        a[5] += (r * nh).sum()
        a[6] += (r * nh ** 2).sum()
        a[7] = max(a[7], nh.max())
    return acc


def summarize(acc: np.ndarray, n_experts: int):
    """(mass [E], phi [S, 3 kinds, 3]) from the accumulators.  Kinds: gate, up (input x), down (input h)."""
    acc = np.asarray(acc, np.float64)
    S = acc.shape[0]
    total = acc[:n_experts, 0].sum()
    mass = acc[:n_experts, 0] / total if total > 0 else np.zeros(n_experts)
    phi = np.zeros((S, 3, 3), np.float64)
    for s in range(S):
        sr = acc[s, 0]
        if sr <= 0:
            continue
        fx = np.array([acc[s, 2] / sr, np.sqrt(acc[s, 3] / sr), acc[s, 4]])
        fh = np.array([acc[s, 5] / sr, np.sqrt(acc[s, 6] / sr), acc[s, 7]])
        phi[s, 0] = fx
        phi[s, 1] = fx
        phi[s, 2] = fh
    return mass, phi
