"""Helpers shared by the GPU parity tests: build a layer on the device, mirror it for the oracle."""
from __future__ import annotations

import numpy as np
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth


def export_to_oracle(ctx, page, orc):
    """Device page (TILED) -> oracle Page (canonical, host numpy), through pw_export_page."""
    ex = ctx.pw_export_page(page)
    torch.cuda.synchronize()
    codes = ex.codes.cpu().numpy()
    ng = page.cols // B.GROUP
    if page.bits == 16:
        return orc.Page(codes, None, None, page.rows, page.cols, 16)
    scales = ex.scales.view(torch.int16).cpu().numpy().view(np.uint16).reshape(page.rows, ng)
    zps = ex.zps.view(torch.int16).cpu().numpy().view(np.uint16).reshape(page.rows, ng)
    return orc.Page(codes, scales, zps, page.rows, page.cols, page.bits)


def import_from_oracle(ctx, opage):
    """Oracle Page -> device page (TILED), through pw_import_page."""
    can = B.Page(opage.rows, opage.cols, opage.bits, ctx.device, B.PW_LAYOUT_CANONICAL)
    can.codes.copy_(torch.from_numpy(opage.codes))
    if opage.bits < 16:
        can.scales.copy_(torch.from_numpy(opage.scales.view(np.float16).reshape(-1)))
        can.zps.copy_(torch.from_numpy(opage.zps.view(np.float16).reshape(-1)))
    return ctx.pw_import_page(can)


def pages_equal(a, b) -> bool:
    if a.bits != b.bits or a.rows != b.rows or a.cols != b.cols:
        return False
    if not np.array_equal(a.codes, b.codes):
        return False
    if a.bits == 16:
        return True
    return np.array_equal(a.scales, b.scales) and np.array_equal(a.zps, b.zps)


def build_layer(ctx, cfg, layer=0, bits=None, device="cuda"):
    """Quantizes every block of one layer on the GPU and publishes the rows.  Returns (pages, bits)."""
    bits = synth.assign_bits(cfg, layer) if bits is None else bits
    S = cfg.n_experts + cfg.n_shared
    pages, entries = [], []
    for e in range(S):
        for u in range(3):
            w = synth.block_weights(cfg, layer, e, u, device=device)
            pg = ctx.pw_quantize_block(w, int(bits[e, u]))
            pages.append(pg)
            entries.append((layer, e, u, pg))
            del w
    ctx.pw_set_page_table(entries)
    return pages, bits


def make_ctx(cfg, max_tokens=None, n_layers=None):
    return B.Context(n_layers or cfg.n_layers, cfg.n_experts, cfg.n_shared, cfg.hidden, cfg.ffn,
                     max_tokens or cfg.tokens, cfg.top_k)


def error_metrics(got: np.ndarray, ref: np.ndarray):
    d = got.astype(np.float64) - ref.astype(np.float64)
    return float(np.abs(d).max()), float(np.linalg.norm(d) / max(np.linalg.norm(ref.astype(np.float64)), 1e-30))
