#!/usr/bin/env python
"""Benchmark of the paged-weight MoE hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One "step" is one layer call of the whole forward path -- page-table commit of a row, router, stable
permutation, page-table lookup, gate/up contraction with in-kernel dequantization, SwiGLU, down
contraction, gate-weighted combine -- on a batch of synthetic decode tokens, with the layer's
mixed-bitwidth weight pages already resident in HBM.  The quantize / demote kernels and their
side-stream overlap with decode are timed in separate, shorter regions of the same run and reported
under "demote"; the prefill configuration under "prefill".  N > 1 runs N independent replicas
(the layer call does not shard and has no collective).

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import re
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2607_16184_b200 import replicas, synth

METRIC = "MoE-layer decode tokens/s & HBM GB/s vs 8 TB/s; prefill TFLOP/s; demote GB/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def profiled_traffic(name: str):
    """(DRAM bytes per launch of the dominant kernel, algorithmic bytes of the same captured launches) from the
    committed ncu summary, or (None, None).  The capture covers one launch per layer the bench rotates over, so
    the two averages are like for like with `algorithmic_bytes_per_launch`."""
    p = os.path.join(ROOT, "profiles", name)
    if not os.path.exists(p):
        return None, None
    txt = open(p).read()
    m = re.search(r"dram_bytes_per_launch_full_size:\s*([0-9.eE+]+)", txt)
    a = re.search(r"algorithmic_bytes_per_launch_of_capture:\s*([0-9.eE+]+)", txt)
    return (float(m.group(1)) if m else None), (float(a.group(1)) if a else None)


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs (read-only NVML queries)."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self._stop = threading.Event()
        self._thread = None
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {}
        for n in dir(nv):
            if n.startswith("nvmlClocksEventReason") or n.startswith("nvmlClocksThrottleReason"):
                v = getattr(nv, n)
                if isinstance(v, int) and v:
                    names[v] = n.replace("nvmlClocksEventReason", "").replace("nvmlClocksThrottleReason", "")
        while not self._stop.is_set():
            try:
                self.samples.append((time.time(), int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))))
                try:
                    bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for v, n in names.items():
                    if bits & v and n not in ("None", "All"):
                        self.reasons.add(n)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        self.t0 = time.time()

    def stop(self):
        self.t1 = time.time()
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=2)
        mhz = [m for (t, m) in self.samples if self.t0 <= t <= self.t1] or [m for (_, m) in self.samples]
        norm = {"SwPowerCap": "sw_power_cap", "HwSlowdown": "hw_slowdown", "HwThermalSlowdown": "hw_thermal_slowdown",
                "SwThermalSlowdown": "sw_thermal_slowdown", "GpuIdle": "gpu_idle",
                "ApplicationsClocksSetting": "applications_clocks_setting", "SyncBoost": "sync_boost",
                "HwPowerBrakeSlowdown": "hw_power_brake_slowdown", "DisplayClockSetting": "display_clock_setting"}
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted({norm.get(r, r) for r in self.reasons} - {"gpu_idle"}), "samples": len(mhz)}


def page_bytes_total(bits_table, cfg, active_mask=None):
    """(gate+up bytes, down bytes) of the pages of the experts that hold at least one token."""
    from paper_2607_16184_b200 import binding as B
    gu = dn = 0
    for e in range(bits_table.shape[0]):
        if active_mask is not None and not active_mask[e]:
            continue
        for u in range(3):
            rows, cols = cfg.block_shape(u)
            n = B.pw_page_bytes(rows, cols, int(bits_table[e, u]))[0]
            if u == 2:
                dn += n
            else:
                gu += n
    return gu, dn


def build_layers(ctx, cfg, n_layers, device, planes_q=0):
    """planes_q: 0 = ordinary pages at the configured bitwidths; 2, 3 or 4 = every routed block is a bit-plane
    block read at that many bits."""
    layers = []
    for layer in range(n_layers):
        bits = synth.assign_bits(cfg, layer)
        if planes_q:
            bits[:cfg.n_experts] = planes_q
        pages, entries = [], []
        for e in range(cfg.n_experts + cfg.n_shared):
            for u in range(3):
                w = synth.block_weights(cfg, layer, e, u, device=device)
                if planes_q and e < cfg.n_experts:
                    pg = ctx.pw_quantize_planes(w).at(planes_q, detach=True)
                else:
                    pg = ctx.pw_quantize_block(w, int(bits[e, u]))
                pages.append(pg)
                entries.append((layer, e, u, pg))
                del w
        ctx.pw_set_page_table(entries)
        layers.append({"bits": bits, "pages": pages, "entries": entries,
                       "x": synth.activations(cfg, layer, device=device),
                       "logits": synth.router_logits(cfg, layer, device=device)})
    torch.cuda.synchronize(device)
    return layers


def time_region(fn, steps, device):
    torch.cuda.synchronize(device)
    replicas.barrier(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        fn(i)
    e1.record()
    torch.cuda.synchronize(device)
    replicas.barrier(device)
    return e0.elapsed_time(e1)


def time_region_chunks(fn, steps, device, chunk=50):
    """time_region with an event every `chunk` steps as well (one event per 50 calls does not disturb the chain):
    returns the total and the per-step times of the chunks, for a median and a best figure."""
    torch.cuda.synchronize(device)
    replicas.barrier(device)
    marks = [torch.cuda.Event(enable_timing=True)]
    marks[0].record()
    for i in range(steps):
        fn(i)
        if (i + 1) % chunk == 0 or i + 1 == steps:
            marks.append(torch.cuda.Event(enable_timing=True))
            marks[-1].record()
    torch.cuda.synchronize(device)
    replicas.barrier(device)
    bounds = [min((j + 1) * chunk, steps) - j * chunk for j in range(len(marks) - 1)]
    per_step = [marks[j].elapsed_time(marks[j + 1]) / n for j, n in enumerate(bounds) if n == chunk]
    return marks[0].elapsed_time(marks[-1]), per_step


def cpu_oracle_sample(cfg, layer_pages_host, x, logits, n_tokens):
    """Times the CPU oracle, as it stands, on the first n_tokens tokens of the batch."""
    from oracle import oracle
    t0 = time.time()
    oracle.moe_forward(x, logits, cfg.top_k, layer_pages_host, n_shared=cfg.n_shared, tokens=list(range(n_tokens)))
    dt = time.time() - t0
    return n_tokens / dt, dt, oracle.num_threads()


def export_layer_to_host(ctx, layer, cfg):
    from oracle import oracle
    out = []
    for pg in layer["pages"]:
        ex = ctx.pw_export_page(pg)
        torch.cuda.synchronize()
        ng = pg.cols // 128
        if pg.bits == 16:
            out.append(oracle.Page(ex.codes.cpu().numpy(), None, None, pg.rows, pg.cols, 16))
        else:
            out.append(oracle.Page(ex.codes.cpu().numpy(),
                                   ex.scales.view(torch.int16).cpu().numpy().view(np.uint16).reshape(pg.rows, ng),
                                   ex.zps.view(torch.int16).cpu().numpy().view(np.uint16).reshape(pg.rows, ng),
                                   pg.rows, pg.cols, pg.bits))
        del ex
    return out


def run_prefill(device, peaks, steps=20, warmup=3):
    """Prefill configuration (4096 tokens, bits from {16,8,4}): useful TFLOP/s of one layer call."""
    from paper_2607_16184_b200 import binding as B
    cfg = synth.CONFIGS["mixtral_prefill"]
    ctx = B.Context(1, cfg.n_experts, cfg.n_shared, cfg.hidden, cfg.ffn, cfg.tokens, cfg.top_k, device=device)
    layer = build_layers(ctx, cfg, 1, device)[0]
    out = torch.empty(cfg.tokens, cfg.hidden, dtype=torch.float32, device=device)
    fn = lambda i: ctx.pw_moe_forward(0, layer["x"], layer["logits"], cfg.top_k, out=out, mode=B.PW_MODE_TENSOR)
    for i in range(warmup):
        fn(i)
    ms = time_region(fn, steps, device) / steps
    status = ctx.pw_last_device_status()
    flops = 2.0 * cfg.tokens * cfg.top_k * 3 * cfg.hidden * cfg.ffn
    tf = flops / (ms * 1e-3) / 1e12
    ctx.close()
    return {"workload": "mixtral_prefill: T=4096, E=8, top-2, H=4096, F=14336, bits iid {16,8,4}", "ms_per_call": ms,
            "tokens_per_s": cfg.tokens / (ms * 1e-3), "tflops": tf, "useful_flop_per_call": flops,
            "frac_of_measured_bf16_burst": tf / peaks["bf16_tflops"],
            "frac_of_measured_bf16_sustained": tf / peaks["bf16_tflops_sustained"],
            "frac_of_nominal_2250": tf / NOMINAL_BF16_TFLOPS, "device_status": status, "steps": steps}


def run_demote(ctx, cfg, layers, device, peaks, decode_fn, decode_ms):
    """pw_demote_block alone (16->4 on distinct fp16 pages, then 4->2) and overlapped with decode on a side stream."""
    from paper_2607_16184_b200 import binding as B
    rows, cols = cfg.block_shape(0)
    n_src = 6                                   # six 117 MB sources: well past L2 between reuses
    srcs = [ctx.pw_quantize_block(synth.block_weights(cfg, 100, e, 0, device=device), 16) for e in range(n_src)]
    dst4 = [B.Page(rows, cols, 4, device) for _ in range(n_src)]
    dst2 = [B.Page(rows, cols, 2, device) for _ in range(n_src)]
    b16, b4, b2 = (B.pw_page_bytes(rows, cols, b)[0] for b in (16, 4, 2))
    for i in range(n_src):
        ctx.pw_demote_block(srcs[i], 4, dst=dst4[i])
        ctx.pw_demote_block(dst4[i], 2, dst=dst2[i])
    reps = 18
    ms164 = time_region(lambda i: ctx.pw_demote_block(srcs[i % n_src], 4, dst=dst4[i % n_src]), reps, device) / reps
    ms42 = time_region(lambda i: ctx.pw_demote_block(dst4[i % n_src], 2, dst=dst2[i % n_src]), reps, device) / reps
    # overlapped: one 16->4 demote per decode step on a side stream (never committed).  Two arrangements: both
    # streams at the default priority, and the decode on a stream of higher priority than the demote's, which is
    # how a server keeps page movement in the gaps of the forward pass (the block scheduler then places a waiting
    # CTA of the forward call before any further CTA of the demote).
    # Blocks of decode steps alone and with the demotes alternate, so that both see the same clocks (a short
    # burst after an idle moment runs at boost clocks, a long loop under the power cap does not).
    def overlapped(main, side):
        n_steps, rounds = 60, 4
        alone_ms = over_ms = side_ms = 0.0
        with torch.cuda.stream(main):
            for _ in range(rounds):
                alone_ms += time_region(decode_fn, n_steps, device)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                side.wait_stream(main)
                e0.record()
                s0.record(side)
                for i in range(n_steps):
                    ctx.pw_demote_block(srcs[i % n_src], 4, dst=dst4[i % n_src], stream=side)
                    decode_fn(i)
                e1.record()
                s1.record(side)
                torch.cuda.synchronize(device)
                over_ms += e0.elapsed_time(e1)
                side_ms += s0.elapsed_time(s1)
        n = rounds * n_steps
        return {"decode_ms_per_step": over_ms / n, "decode_ms_alone": alone_ms / n,
                "decode_slowdown": 1.0 - alone_ms / over_ms if over_ms > 0 else None,
                "demote_16to4_gbs_side_stream": (b16 + b4) / (side_ms / n * 1e-3) / 1e9, "steps": n}

    cur = torch.cuda.current_stream(device)
    cur.synchronize()
    under_default = overlapped(cur, torch.cuda.Stream(device=device))
    hp = torch.cuda.Stream(device=device, priority=-1)
    hp.wait_stream(cur)
    under_prio = overlapped(hp, torch.cuda.Stream(device=device, priority=0))
    cur.wait_stream(hp)
    gbs = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9
    return {"block": "%dx%d" % (rows, cols),
            "16to4": {"ms": ms164, "gbs": gbs(b16 + b4, ms164), "frac_of_measured_hbm": gbs(b16 + b4, ms164) / peaks["hbm_gbs"],
                      "frac_of_nominal_8000": gbs(b16 + b4, ms164) / NOMINAL_HBM_GBS, "bytes": b16 + b4},
            "4to2": {"ms": ms42, "gbs": gbs(b4 + b2, ms42), "frac_of_measured_hbm": gbs(b4 + b2, ms42) / peaks["hbm_gbs"],
                     "frac_of_nominal_8000": gbs(b4 + b2, ms42) / NOMINAL_HBM_GBS, "bytes": b4 + b2},
            "under_decode": under_prio, "under_decode_equal_priorities": under_default}


def run_residency(ctx, cfg, layers, device, decode_fn, decode_ms):
    """pw_offload_page / pw_reload_page of 16-bit blocks (rows whose committed bitwidth is lower): each direction
    alone, against a plain pinned copy of the same size, and both directions on a side stream under decode."""
    from paper_2607_16184_b200 import binding as B
    rows, cols = cfg.block_shape(0)
    nbytes = B.pw_page_bytes(rows, cols, 16)[0]
    bits = layers[0]["bits"]
    targets = [(0, e, u) for e in range(cfg.n_experts) for u in (0, 1) if int(bits[e, u]) != 16][:6]
    if not targets:
        return None
    page = ctx.pw_quantize_block(synth.block_weights(cfg, 200, 0, 0, device=device), 16)
    hosts = [torch.empty(nbytes, dtype=torch.uint8).pin_memory() for _ in targets]
    side = torch.cuda.Stream(device=device)
    gbs = lambda b, ms: b / (ms * 1e-3) / 1e9

    def timed_side(fn):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(device)
        a.record(side)
        fn()
        b.record(side)
        side.synchronize()
        return a.elapsed_time(b)

    # the link itself: the same bytes with a plain asynchronous copy
    with torch.cuda.stream(side):
        ms_d2h = timed_side(lambda: [hosts[i].copy_(page.codes, non_blocking=True) for i in range(len(targets))])
        ms_h2d = timed_side(lambda: [page.codes.copy_(hosts[i], non_blocking=True) for i in range(len(targets))])
    ms_off = timed_side(lambda: [ctx.pw_offload_page(*t, page, stream=side, host=hosts[i]) for i, t in enumerate(targets)])
    assert all(ctx.pw_page_state(*t, 16) == B.PW_STATE_CPU_RESIDENT for t in targets)
    back = []
    ms_rel = timed_side(lambda: back.extend(ctx.pw_reload_page(*t, 16, hosts[i], stream=side) for i, t in enumerate(targets)))
    assert all(ctx.pw_page_state(*t, 16) == B.PW_STATE_GPU_RESIDENT for t in targets)
    assert torch.equal(back[-1].codes, page.codes)
    total = nbytes * len(targets)
    # under decode: every step one page moves (out if it is resident, back in if it is away), on the side stream
    # (blocks alone and with page movement alternate, so that both see the same clocks)
    n_steps, rounds, moved = 60, 4, 0
    alone_ms = over_ms = ms_side = 0.0
    for _ in range(rounds):
        alone_ms += time_region(decode_fn, n_steps, device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        s0.record(side)
        for i in range(n_steps):
            j = i % len(targets)
            st = ctx.pw_page_state(*targets[j], 16)
            if st == B.PW_STATE_GPU_RESIDENT:
                ctx.pw_offload_page(*targets[j], back[j], stream=side, host=hosts[j])
                moved += nbytes
            elif st == B.PW_STATE_CPU_RESIDENT:
                back[j] = ctx.pw_reload_page(*targets[j], 16, hosts[j], stream=side)
                moved += nbytes
            decode_fn(i)
        e1.record()
        s1.record(side)
        torch.cuda.synchronize(device)
        over_ms += e0.elapsed_time(e1)
        ms_side += s0.elapsed_time(s1)
    decode_ms = alone_ms / (rounds * n_steps)
    ms_dec = over_ms / (rounds * n_steps)
    n_steps *= rounds
    for t in targets:                                  # leave no record behind for the rest of the run
        if ctx.pw_page_state(*t, 16) != B.PW_STATE_IN_TRANSFER:
            ctx.pw_drop_page(*t, 16)
    return {"block": "%dx%d at 16 bits, %d bytes, %d pages per measurement" % (rows, cols, nbytes, len(targets)),
            "offload_gbs": gbs(total, ms_off), "reload_gbs": gbs(total, ms_rel),
            "plain_copy_d2h_gbs": gbs(total, ms_d2h), "plain_copy_h2d_gbs": gbs(total, ms_h2d),
            "under_decode": {"decode_ms_per_step": ms_dec, "decode_ms_alone": decode_ms,
                             "decode_slowdown": 1.0 - decode_ms / ms_dec if ms_dec > 0 else None,
                             "moved_gbs_side_stream": gbs(moved, ms_side), "moved_bytes": moved,
                             "steps": n_steps}}


def algorithmic_bytes(ctx, cfg, layers, out, mode):
    """(gate+up page bytes, down page bytes) of the experts that hold tokens, averaged over the layers."""
    T, k, L = cfg.tokens, cfg.top_k, len(layers)
    gu_bytes = dn_bytes = 0.0
    for li, lay in enumerate(layers):
        ctx.pw_moe_forward(li, lay["x"], lay["logits"], k, out=out, mode=mode)
        counts = ctx.pw_get_routing(T, k)["counts"].cpu().numpy()
        active = np.concatenate([counts > 0, np.ones(cfg.n_shared, bool)])
        gu, dn = page_bytes_total(lay["bits"], cfg, active)
        gu_bytes += gu / L
        dn_bytes += dn / L
    return gu_bytes, dn_bytes


def kernel_pass(ctx, step, steps, device):
    """Per-kernel device times of the same loop: events recorded around every kernel of the call."""
    ctx.pw_kernel_timing(True)
    ms = time_region(step, steps, device)
    ktimes, kcalls = ctx.pw_get_kernel_times()
    ctx.pw_kernel_timing(False)
    return {n: v / max(kcalls, 1) for n, v in ktimes.items()}, ms / steps


def decode_workload(device, peaks, cfg, L, mode, steps, warmup, min_seconds=0.6, planes_q=0):
    """One decode configuration in a context of its own: step time, per-kernel times and roofline fractions of a
    region of at least `min_seconds` of back-to-back steps (sampled clocks), rotating over L distinct layers."""
    from paper_2607_16184_b200 import binding as B
    ctx = B.Context(L, cfg.n_experts, cfg.n_shared, cfg.hidden, cfg.ffn, cfg.tokens, cfg.top_k, device=device)
    layers = build_layers(ctx, cfg, L, device, planes_q)
    T, k = cfg.tokens, cfg.top_k
    out = torch.empty(T, cfg.hidden, dtype=torch.float32, device=device)

    def step(i):
        lay = layers[i % L]
        ctx.pw_set_page_table(lay["entries"][(i // L) % len(lay["entries"]):][:1])
        ctx.pw_moe_forward(i % L, lay["x"], lay["logits"], k, out=out, mode=mode)

    for i in range(max(warmup, 3)):
        step(i)
    ms_probe = time_region(step, max(steps, 20), device) / max(steps, 20)
    n = max(steps, int(np.ceil(min_seconds / (ms_probe * 1e-3))))
    sampler = ClockSampler(device.index or 0)
    sampler.start()
    ms_step = time_region(step, n, device) / n
    clocks = sampler.stop()
    kavg, _ = kernel_pass(ctx, step, n, device)
    status = ctx.pw_last_device_status()
    gu_bytes, dn_bytes = algorithmic_bytes(ctx, cfg, layers, out, mode)
    R = T * k + cfg.n_shared * T
    io_bytes = 2 * T * cfg.hidden + 4 * T * cfg.n_experts + 4 * T * cfg.hidden
    call_bytes = gu_bytes + dn_bytes + io_bytes
    gbs = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0
    gu_gbs = gbs(gu_bytes + 2.0 * R * cfg.hidden, kavg["ffn_gate_up"])
    dn_gbs = gbs(dn_bytes + 2.0 * R * cfg.ffn, kavg["ffn_down"])
    res = {"workload": "%s: E=%d+%d top-%d H=%d F=%d T=%d, %s routing, bit rule %s, %d layers of %.3f GB of pages"
                       % (cfg.name, cfg.n_experts, cfg.n_shared, k, cfg.hidden, cfg.ffn, T, cfg.routing, cfg.bit_rule, L,
                          (gu_bytes + dn_bytes) / 1e9),
           "steps": n, "ms_per_step": ms_step, "tokens_per_s": T / (ms_step * 1e-3), "sm_mhz": clocks["sm_mhz"],
           "reasons": clocks["reasons"], "algorithmic_bytes_per_call": call_bytes,
           "forward_gbs": gbs(call_bytes, ms_step), "forward_frac": gbs(call_bytes, ms_step) / peaks["hbm_gbs"],
           "gate_up_ms": kavg["ffn_gate_up"], "gate_up_gbs": gu_gbs, "gate_up_frac": gu_gbs / peaks["hbm_gbs"],
           "down_ms": kavg["ffn_down"], "down_gbs": dn_gbs, "down_frac": dn_gbs / peaks["hbm_gbs"],
           "small_kernels_ms": sum(v for n_, v in kavg.items() if not n_.startswith("ffn")),
           "device_status": status}
    ctx.close()
    del layers, ctx
    torch.cuda.empty_cache()
    return res


def run_gpu(args):
    from paper_2607_16184_b200 import binding as B
    from paper_2607_16184_b200 import build as pwbuild
    rank, local_rank, world = replicas.init("nccl")
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    device = torch.device("cuda", local_rank if world > 1 else 0)
    torch.cuda.set_device(device)
    if rank == 0:
        pwbuild.build()
    replicas.barrier(device)
    peaks = measured_peaks()
    if args.only == "prefill":
        print(json.dumps({"metric": "prefill TFLOP/s", "data": "synthetic",
                          "prefill": run_prefill(device, peaks, steps=min(args.steps, 20), warmup=3)}))
        return
    cfg = synth.CONFIGS[args.config]
    if args.uniform_bits:
        import dataclasses
        cfg = dataclasses.replace(cfg, bit_rule="uniform%d" % args.uniform_bits)
    L = args.layers or (8 if cfg.name in ("latency_b1", "latency_b4", "manyexpert_decode") else 3)
    ctx = B.Context(L, cfg.n_experts, cfg.n_shared, cfg.hidden, cfg.ffn, cfg.tokens, cfg.top_k, device=device)
    layers = build_layers(ctx, cfg, L, device)
    T, k = cfg.tokens, cfg.top_k
    out = torch.empty(T, cfg.hidden, dtype=torch.float32, device=device)
    mode = {"auto": B.PW_MODE_AUTO, "tensor": B.PW_MODE_TENSOR, "simt": B.PW_MODE_SIMT}[args.mode]

    def step(i):
        lay = layers[i % L]
        ctx.pw_set_page_table(lay["entries"][(i // L) % len(lay["entries"]):][:1])      # commit one row (S10)
        ctx.pw_moe_forward(i % L, lay["x"], lay["logits"], k, out=out, mode=mode)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize(device)
    if args.only == "demote":
        ms_alone = time_region(step, 30, device) / 30
        print(json.dumps({"metric": "demote GB/s", "data": "synthetic",
                          "demote": run_demote(ctx, cfg, layers, device, peaks, step, ms_alone)}))
        return
    sampler = ClockSampler(device.index or 0)
    n0 = ctx.pw_launch_count()
    sampler.start()
    ms_total = time_region(step, args.steps, device)
    clocks = sampler.stop()
    launches = ctx.pw_launch_count() - n0
    status = ctx.pw_last_device_status()
    ms_max, tokens_all = replicas.aggregate(ms_total, float(T * args.steps), device)
    value = tokens_all / (ms_max * 1e-3)

    # per-kernel device times, same loop, events recorded around every kernel of the call
    kavg, ms_timed_step = kernel_pass(ctx, step, args.steps, device)

    # algorithmic bytes of a layer call: pages of experts that hold tokens + activations in/out
    gu_bytes, dn_bytes = algorithmic_bytes(ctx, cfg, layers, out, mode)
    R = T * k + cfg.n_shared * T
    io_bytes = 2 * T * cfg.hidden + 4 * T * cfg.n_experts + 4 * T * cfg.hidden
    call_bytes = gu_bytes + dn_bytes + io_bytes
    ms_step = ms_max / args.steps
    gu_kernel_bytes = gu_bytes + 2.0 * R * cfg.hidden           # pages + the gathered fp16 token rows it reads
    gbs = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0
    gu_gbs = gbs(gu_kernel_bytes, kavg["ffn_gate_up"])
    dn_gbs = gbs(dn_bytes + 2.0 * R * cfg.ffn, kavg["ffn_down"])
    traffic, traffic_alg = (profiled_traffic("ffn_gate_up_mixtral_decode.md")
                            if cfg.name == "mixtral_decode" and not args.uniform_bits else (None, None))
    roofline = {"bound": "hbm", "kernel": "ffn_tc_kernel<0> (gate/up + SwiGLU)", "achieved": gu_gbs,
                "peak": peaks["hbm_gbs"], "peak_source": peaks["source"], "unit": "GB/s",
                "frac": gu_gbs / peaks["hbm_gbs"], "frac_of_nominal_8000": gu_gbs / NOMINAL_HBM_GBS,
                "algorithmic_bytes_per_launch": gu_kernel_bytes, "avg_launch_ms": kavg["ffn_gate_up"],
                "traffic": traffic, "traffic_capture_algorithmic_bytes": traffic_alg}

    # Steady state: whatever --steps was, at least 0.6 s of back-to-back steps with the clocks sampled (a short
    # region right after an idle moment runs at boost clocks; a serving loop runs under the power cap), then the
    # per-kernel pass of the same length.
    n_steady = max(args.steps, int(np.ceil(args.steady_seconds / (ms_step * 1e-3))))
    sampler2 = ClockSampler(device.index or 0)
    sampler2.start()
    ms_steady_total, chunk_ms = time_region_chunks(step, n_steady, device)
    ms_steady = ms_steady_total / n_steady
    clocks2 = sampler2.stop()
    kavg2, _ = kernel_pass(ctx, step, n_steady, device)
    steady = {"steps": n_steady, "ms_per_step": ms_steady, "tokens_per_s": T / (ms_steady * 1e-3),
              "median_ms_per_step": float(np.median(chunk_ms)) if chunk_ms else None,      # over chunks of 50 steps
              "best_ms_per_step": float(np.min(chunk_ms)) if chunk_ms else None,
              "sm_mhz": clocks2["sm_mhz"], "reasons": clocks2["reasons"],
              "roofline_frac": gbs(gu_kernel_bytes, kavg2["ffn_gate_up"]) / peaks["hbm_gbs"],
              "gate_up_ms": kavg2["ffn_gate_up"], "down_ms": kavg2["ffn_down"],
              "down_frac": gbs(dn_bytes + 2.0 * R * cfg.ffn, kavg2["ffn_down"]) / peaks["hbm_gbs"],
              "forward_frac": gbs(call_bytes, ms_steady) / peaks["hbm_gbs"],
              "forward_frac_of_nominal_8000": gbs(call_bytes, ms_steady) / NOMINAL_HBM_GBS}

    # end to end: host buffers in, host buffer out, through the host-buffer entry point
    xh = [lay["x"].cpu().pin_memory() for lay in layers]
    lh = [lay["logits"].cpu().pin_memory() for lay in layers]
    oh = torch.empty(T, cfg.hidden, dtype=torch.float32).pin_memory()

    def step_e2e(i):
        lay = layers[i % L]
        ctx.pw_set_page_table(lay["entries"][(i // L) % len(lay["entries"]):][:1])
        ctx.pw_moe_forward_host(i % L, xh[i % L], lh[i % L], k, oh, mode=mode)

    for i in range(3):
        step_e2e(i)
    ms_e2e = time_region(step_e2e, args.steps, device)
    ms_e2e_max, tok_e2e = replicas.aggregate(ms_e2e, float(T * args.steps), device)
    e2e = {"value": tok_e2e / (ms_e2e_max * 1e-3), "unit": "tokens/s",
           "h2d_bytes_per_step": int(xh[0].numel() * 2 + lh[0].numel() * 4), "d2h_bytes_per_step": int(oh.numel() * 4)}

    line = {"metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": "%s: one MoE layer call, E=%d top-%d H=%d F=%d T=%d, %s routing, bit mix %s; "
                                   "rotating over %d distinct layers (%.2f GB of pages each, larger than L2)"
                                   % (cfg.name, cfg.n_experts, k, cfg.hidden, cfg.ffn, T, cfg.routing, cfg.bit_rule, L,
                                      (gu_bytes + dn_bytes) / 1e9),
                       "mode": args.mode, "l2": "inputs larger than L2", "replicas": world,
                       "bits_realised": {str(b): int((np.stack([l["bits"] for l in layers]) == b).sum()) for b in synth.BITS}},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "device_status": status,
            "roofline": roofline, "steady": steady,
            "forward": {"algorithmic_bytes_per_call": call_bytes, "hbm_gbs": gbs(call_bytes, ms_step),
                        "frac_of_measured_hbm": gbs(call_bytes, ms_step) / peaks["hbm_gbs"],
                        "frac_of_nominal_8000": gbs(call_bytes, ms_step) / NOMINAL_HBM_GBS,
                        "kernel_ms": kavg, "kernel_timed_ms_per_step": ms_timed_step,
                        "ffn_down_gbs": dn_gbs}}

    if rank == 0 and world == 1 and not args.skip_extra:
        # observation taps (routing mass, routed-input features): the same timed loop with the taps on
        ctx.pw_observe(True)
        for i in range(3):
            step(i)
        ms_obs = time_region(step, args.steps, device) / args.steps
        ctx.pw_kernel_timing(True)
        time_region(step, args.steps, device)
        kt, kc = ctx.pw_get_kernel_times()
        ctx.pw_kernel_timing(False)
        mass, _ = ctx.pw_observation_summary(0)
        R = T * k + cfg.n_shared * T
        line["observe"] = {"ms_per_step_taps_on": ms_obs, "ms_per_step_taps_off": ms_step,
                           "taps_kernels_ms": kt["observe"] / max(kc, 1),
                           "bytes_read_per_call": 2.0 * R * (cfg.hidden + cfg.ffn),
                           "mass_layer0_sum": float(mass.sum().item())}
        ctx.pw_observe(False)
        # the same step with each layer's forward call replayed from a CUDA graph (the commit stays eager)
        graphs = []
        torch.cuda.synchronize(device)
        for li, lay in enumerate(layers if not args.skip_graph else []):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                ctx.pw_moe_forward(li, lay["x"], lay["logits"], k, out=out, mode=mode)
            graphs.append(g)

        def step_graph(i):
            lay = layers[i % L]
            ctx.pw_set_page_table(lay["entries"][(i // L) % len(lay["entries"]):][:1])
            graphs[i % L].replay()

        if graphs:
            for i in range(3):
                step_graph(i)
            ms_graph = time_region(step_graph, args.steps, device) / args.steps
            line["cuda_graph"] = {"ms_per_step": ms_graph, "tokens_per_s": T / (ms_graph * 1e-3),
                                  "ms_per_step_eager": ms_step}
        del graphs
        line["demote"] = run_demote(ctx, cfg, layers, device, peaks, step, ms_step)
        line["residency"] = run_residency(ctx, cfg, layers, device, step, ms_step)
        line["prefill"] = run_prefill(device, peaks)     # its own context and pages (about 2 GB more)
        if cfg.name == "mixtral_decode" and not args.uniform_bits:
            # does a demote buy time?  the gate/up and down kernels on tables of one bitwidth each
            import dataclasses
            per_bits = {}
            for b in synth.BITS:
                r = decode_workload(device, peaks, dataclasses.replace(cfg, bit_rule="uniform%d" % b), 1, mode, 100, 3,
                                    min_seconds=0.15)
                per_bits[str(b)] = {key: r[key] for key in ("ms_per_step", "gate_up_ms", "gate_up_gbs", "gate_up_frac",
                                                             "down_ms", "down_gbs", "down_frac", "forward_frac",
                                                             "sm_mhz")}
                per_bits[str(b)]["gate_up_tiles_per_s"] = (2.0 * cfg.n_experts * (cfg.ffn // 128) * (cfg.hidden // 128)
                                                           / (r["gate_up_ms"] * 1e-3))
            line["per_bits"] = per_bits
            # the same layer with every routed block held as overlaid bit-planes and read at 4, 3 and 2 bits
            planes = {}
            keys = ("ms_per_step", "gate_up_ms", "gate_up_gbs", "gate_up_frac", "down_ms", "down_gbs", "down_frac",
                    "forward_frac", "sm_mhz")
            for q in (4, 3, 2):
                r = decode_workload(device, peaks, dataclasses.replace(cfg, bit_rule="all16"), 1, mode, 100, 3,
                                    min_seconds=0.15, planes_q=q)
                planes[str(q)] = {key: r[key] for key in keys}
            line["bit_planes"] = planes
            # the other decode configuration (64 routed top-6 + 2 shared experts, batch 256)
            line["finegrained_decode"] = decode_workload(device, peaks, synth.CONFIGS["finegrained_decode"], 6, mode,
                                                         200, 5)
    # (the CPU oracle runs after the GPU extras: its OpenMP threads keep the host cores busy for a while
    # afterwards, and the extras' launch loops must not compete with them)
    if rank == 0 and world == 1 and not args.skip_cpu:
        # the oracle as it stands, on the same steps the GPU loop rotates over: one call per layer copy, until
        # about --cpu-seconds of CPU time have been spent (at least one call)
        n_tok, dt_all, cores, calls = 0, 0.0, 0, 0
        while dt_all < args.cpu_seconds and calls < 4 * L:
            lay = layers[calls % L]
            host_pages = export_layer_to_host(ctx, lay, cfg)
            v, dt, cores = cpu_oracle_sample(cfg, host_pages, lay["x"].cpu().numpy(), lay["logits"].cpu().numpy(),
                                             min(args.cpu_tokens, T))
            del host_pages
            n_tok += min(args.cpu_tokens, T)
            dt_all += dt
            calls += 1
        line["cpu_baseline"] = {"value": n_tok / dt_all, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                                "sample": "%d layer calls of %d of the %d tokens each, %.1f s of oracle time"
                                          % (calls, min(args.cpu_tokens, T), T, dt_all)}
    else:
        line["cpu_baseline"] = None
    if rank == 0 and world == 1 and not args.skip_extra and cfg.name == "mixtral_decode" and not args.uniform_bits:
        # the fifth configuration at full size, when the device has the memory for it (90 GB of pages)
        ctx.close()
        del layers, ctx, xh, lh
        torch.cuda.empty_cache()
        free, _ = torch.cuda.mem_get_info(device)
        if free >= 110e9:
            d5 = measure_d5(device, peaks, parity_pages=2)
            line["demote_under_load"] = {"workload": d5["config"]["workload"], "tokens_per_s": d5["value"],
                                         "ms_per_step": d5["ms_per_step"], "roofline_frac_all_16bit": d5["roofline"]["frac"],
                                         "d5": d5["d5"], "device_status": d5["device_status"], "clocks": d5["clocks"]}
        else:
            line["demote_under_load"] = {"skipped": "%.0f GB of device memory free, 110 GB needed" % (free / 1e9)}
    if rank == 0:
        print(json.dumps(line))
    replicas.shutdown()


def check_pages_against_oracle(ctx, cfg, pages, keys, chain):
    """A checking leg, not part of the timed path: the committed pages `keys` compared bit for bit with the CPU
    oracle's quantize / demote chain on the regenerated weights.  Returns the number of pages that matched."""
    from oracle import oracle
    oracle.build()
    ok = 0
    for key in keys:
        w = synth.block_weights(cfg, *key, device=ctx.device).cpu().numpy()   # the same draw as the page's
        op = oracle.quantize_block(w, 16)
        for b in chain:
            op = oracle.demote_block(op, b)
        ex = ctx.pw_export_page(pages[key])
        torch.cuda.synchronize()
        ng = pages[key].cols // 128
        same = ex.bits == op.bits and np.array_equal(ex.codes.cpu().numpy(), op.codes)
        if same and op.bits < 16:
            same = (np.array_equal(ex.scales.view(torch.int16).cpu().numpy().view(np.uint16).reshape(-1, ng), op.scales)
                    and np.array_equal(ex.zps.view(torch.int16).cpu().numpy().view(np.uint16).reshape(-1, ng), op.zps))
        ok += int(bool(same))
        del ex, op
    return ok


def measure_d5(device, peaks, parity_pages=4):
    """The demotion-under-load configuration at full size: 32 stacked Mixtral-shaped layers, all 16-bit at the
    start (90 GB of pages), a seeded third of the blocks demoted 16->4 and then 4->2 on a side stream while
    batch-64 decode steps (one call per layer) keep running.  Three runs: decode alone; "shadow" (demotes run
    but are never committed: pure interference); "committed" (every finished demote is published at the next
    call boundary and the page it replaces is released).  Afterwards a seeded sample of the committed pages is
    compared with the oracle's chain."""
    from paper_2607_16184_b200 import binding as B
    cfg = synth.CONFIGS["demote_under_load"]
    T, k = cfg.tokens, cfg.top_k
    per_layer = sum(B.pw_page_bytes(*cfg.block_shape(u), 16)[0] for u in range(3)) * cfg.n_experts
    free, _ = torch.cuda.mem_get_info(device)
    L = int(min(cfg.n_layers, (free - 14e9) // (per_layer * 1.1)))          # demoted copies add < 10 %
    if L < 2:
        raise RuntimeError("not enough free device memory for two layers of %.1f GB" % (per_layer / 1e9))
    ctx = B.Context(L, cfg.n_experts, cfg.n_shared, cfg.hidden, cfg.ffn, T, k, device=device)
    pages, xs, lgs = {}, [], []
    for layer in range(L):
        ents = []
        for e in range(cfg.n_experts):
            for u in range(3):
                w = synth.block_weights(cfg, layer, e, u, device=device)
                pages[(layer, e, u)] = ctx.pw_quantize_block(w, 16)
                ents.append((layer, e, u, pages[(layer, e, u)]))
                del w
        ctx.pw_set_page_table(ents)
        xs.append(synth.activations(cfg, layer, device=device))
        lgs.append(synth.router_logits(cfg, layer, device=device))
    torch.cuda.synchronize(device)
    sched = [key for key in synth.demote_schedule(cfg) if key[0] < L]
    out = torch.empty(T, cfg.hidden, dtype=torch.float32, device=device)
    # forward calls on a stream of higher priority than the demotes' (page movement takes the gaps)
    boot = torch.cuda.current_stream(device)
    main = torch.cuda.Stream(device=device, priority=-1)
    main.wait_stream(boot)
    torch.cuda.set_stream(main)
    side = torch.cuda.Stream(device=device, priority=0)

    def decode_step():
        for layer in range(L):
            ctx.pw_moe_forward(layer, xs[layer], lgs[layer], k, out=out)

    def timed(fn, n):
        torch.cuda.synchronize(device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n):
            fn(i)
        e1.record()
        torch.cuda.synchronize(device)
        return e0.elapsed_time(e1)

    for _ in range(2):
        decode_step()
    sampler = ClockSampler(0)
    sampler.start()
    n0 = ctx.pw_launch_count()
    n_base = 6
    ms_base = timed(lambda i: decode_step(), n_base) / n_base

    # shadow run: one chunk of 16->4 demotes per decode step into a small pool of scratch pages, never committed
    per_step = 8
    rows_cols = [cfg.block_shape(u) for u in range(3)]
    pool = {u: [B.Page(rows_cols[u][0], rows_cols[u][1], 4, device) for _ in range(per_step)] for u in range(3)}
    n_shadow = min(12, max(1, len(sched) // per_step))
    moved = [0]

    def shadow_step(i):
        side.wait_stream(main)
        used = {0: 0, 1: 0, 2: 0}
        for key in sched[i * per_step:(i + 1) * per_step]:
            u = key[2]
            ctx.pw_demote_block(pages[key], 4, dst=pool[u][used[u] % per_step], stream=side)
            used[u] += 1
            moved[0] += B.pw_page_bytes(*rows_cols[u], 16)[0] + B.pw_page_bytes(*rows_cols[u], 4)[0]
        decode_step()

    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(device)
    s0.record(side)
    ms_shadow = timed(shadow_step, n_shadow) / n_shadow
    s1.record(side)
    torch.cuda.synchronize(device)
    shadow_side_ms = s0.elapsed_time(s1)
    shadow_gbs = moved[0] / (shadow_side_ms * 1e-3) / 1e9
    del pool

    # committed run: phase 1 (16->4) then phase 2 (4->2) over the same blocks
    def page_total():
        return sum(B.pw_page_bytes(p.rows, p.cols, p.bits)[0] for p in pages.values())

    bytes_start = page_total()
    phases = []
    for dst_bits in (4, 2):
        todo = list(sched)
        inflight = []
        steps = 0
        moved_b = 0
        torch.cuda.synchronize(device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        while todo or inflight:
            done = [x for x in inflight if x[2].query()]
            if done:
                for key, pg, ev in done:
                    main.wait_event(ev)
                    # The page it replaces is released here.  Its last readers are already enqueued on the main
                    # stream, and whoever gets its memory next (a demote destination, written on the side stream)
                    # starts only after side.wait_stream(main) below.
                    pages[key] = pg
                ctx.pw_set_page_table([(key[0], key[1], key[2], pg) for key, pg, _ in done])
                inflight = [x for x in inflight if not any(x is d for d in done)]
            side.wait_stream(main)
            for key in todo[:per_step]:
                src = pages[key]
                dst = ctx.pw_demote_block(src, dst_bits, stream=side)
                ev = torch.cuda.Event()
                ev.record(side)
                inflight.append((key, dst, ev))
                moved_b += B.pw_page_bytes(src.rows, src.cols, src.bits)[0] + B.pw_page_bytes(src.rows, src.cols, dst_bits)[0]
            todo = todo[per_step:]
            decode_step()
            steps += 1
        e1.record()
        torch.cuda.synchronize(device)
        ms = e0.elapsed_time(e1)
        phases.append({"dst_bits": dst_bits, "blocks": len(sched), "decode_steps": steps, "ms": ms,
                       "tokens_per_s": T * steps / (ms * 1e-3), "demote_bytes_moved": moved_b,
                       "demote_gbs_over_phase": moved_b / (ms * 1e-3) / 1e9, "page_bytes_after": page_total()})
    clocks = sampler.stop()
    launches = ctx.pw_launch_count() - n0
    status = ctx.pw_last_device_status()
    tot_steps = sum(p["decode_steps"] for p in phases)
    tot_ms = sum(p["ms"] for p in phases)
    tok_base = T / (ms_base * 1e-3)
    line = {"metric": METRIC, "value": T * tot_steps / (tot_ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
            "steps": tot_steps, "warmup": 2, "ms_per_step": tot_ms / tot_steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": "demote_under_load: %d stacked layers (E=8 top-2 H=4096 F=14336, T=64), all 16-bit at "
                                   "the start (%.1f GB of pages); a step = one forward call per layer; %d blocks demoted "
                                   "16->4 then 4->2 on a side stream, %d per step, committed between calls"
                                   % (L, bytes_start / 1e9, len(sched), per_step),
                       "l2": "inputs larger than L2", "layers": L, "layers_of_config": cfg.n_layers},
            "clocks": clocks, "e2e": None, "gpu_launches": int(launches), "device_status": status,
            "roofline": {"bound": "hbm", "kernel": "whole decode step, all 16-bit", "unit": "GB/s",
                         "achieved": (L * per_layer) / (ms_base * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                         "peak_source": peaks["source"],
                         "frac": (L * per_layer) / (ms_base * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None},
            "cpu_baseline": None,
            "d5": {"baseline": {"ms_per_step": ms_base, "tokens_per_s": tok_base},
                   "shadow": {"ms_per_step": ms_shadow, "tokens_per_s": T / (ms_shadow * 1e-3),
                              "slowdown": 1.0 - ms_base / ms_shadow, "demotes_per_step": per_step,
                              "demote_gbs_side_stream": shadow_gbs},
                   "committed": phases, "page_bytes_start": bytes_start}}
    picks = [sched[i] for i in np.random.default_rng(11).choice(len(sched), size=min(parity_pages, len(sched)),
                                                                replace=False)] if parity_pages else []
    matched = check_pages_against_oracle(ctx, cfg, pages, picks, (4, 2))
    line["d5"]["parity_checked_pages"] = len(picks)
    line["d5"]["parity_matched_pages"] = matched
    torch.cuda.synchronize(device)
    torch.cuda.set_stream(boot)
    ctx.close()
    return line


def run_d5(args):
    from paper_2607_16184_b200 import build as pwbuild
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    pwbuild.build()
    print(json.dumps(measure_d5(device, measured_peaks())), flush=True)


def run_reference(args):
    """The CPU oracle as the reference arm: the same configuration and metric, each step one whole layer call
    (all tokens of the batch) of the oracle as it stands, on the host cores."""
    rank, _, world = replicas.env_world()
    if rank != 0:
        return
    from oracle import oracle
    oracle.build()
    cfg = synth.CONFIGS[args.config]
    n_tok = cfg.tokens if args.ref_tokens <= 0 else min(args.ref_tokens, cfg.tokens)
    x = synth.activations(cfg, 0).numpy()
    logits = synth.router_logits(cfg, 0).numpy()
    bits = synth.assign_bits(cfg, 0)
    ids, _ = oracle.router(logits, cfg.top_k)
    need = set(int(e) for e in ids[:n_tok].reshape(-1)) | set(range(cfg.n_experts, cfg.n_experts + cfg.n_shared))
    pages = []
    for e in range(cfg.n_experts + cfg.n_shared):
        for u in range(3):
            rows, cols = cfg.block_shape(u)
            if e in need:
                pages.append(oracle.quantize_block(synth.block_weights(cfg, 0, e, u).numpy(), int(bits[e, u])))
            else:   # never read: no token of the step is routed here
                pages.append(oracle.Page(np.zeros(16, np.uint8), None, None, rows, cols, 16))
    toks = list(range(n_tok))
    run = lambda: oracle.moe_forward(x, logits, cfg.top_k, pages, n_shared=cfg.n_shared, tokens=toks)
    for _ in range(args.warmup):
        run()
    t0 = time.time()
    for _ in range(args.steps):
        run()
    dt = time.time() - t0
    v = n_tok * args.steps / dt
    cores = oracle.num_threads()
    same = n_tok == cfg.tokens
    sample = ("whole layer calls of layer 0, all %d tokens per step" % cfg.tokens) if same else \
             ("first %d of %d tokens of layer 0 per step" % (n_tok, cfg.tokens))
    print(json.dumps({"impl": "reference", "metric": METRIC, "value": v, "unit": "tokens/s", "n_gpus": world,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                      "data": "synthetic", "same_config": same,
                      "config": {"workload": "%s (CPU oracle, %s)" % (cfg.name, sample)},
                      "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
                      "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                      "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="mixtral_decode", choices=["mixtral_decode", "finegrained_decode", "demote_under_load", "latency_b1", "latency_b4",
                             "manyexpert_decode"])
    ap.add_argument("--layers", type=int, default=0,
                    help="distinct layer copies the decode loop rotates over (default: 3, or 8 for the small-batch "
                         "configurations, whose calls read less than the L2 holds)")
    ap.add_argument("--mode", default="auto", choices=["auto", "tensor", "simt"])
    ap.add_argument("--cpu-tokens", type=int, default=64)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="oracle time to spend on the cpu_baseline sample")
    ap.add_argument("--ref-tokens", type=int, default=0,
                    help="reference arm: tokens of the batch per step (0 = the whole batch, the configuration itself)")
    ap.add_argument("--uniform-bits", type=int, default=0, choices=[0, 16, 8, 4, 3, 2],
                    help="diagnostic: give every routed block this bitwidth instead of the configured mix")
    ap.add_argument("--steady-seconds", type=float, default=0.6,
                    help="least duration of the steady-state region (0: just --steps steps, for profiler captures)")
    ap.add_argument("--only", default="", choices=["", "prefill", "demote"],
                    help="run one of the extra regions alone and print it (small commands for profiler captures)")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-extra", action="store_true")
    ap.add_argument("--skip-graph", action="store_true", help="leave out the CUDA-graph replay of the step")
    args = ap.parse_args()
    if args.impl == "reference":
        # a whole layer call of the oracle takes about 2 s on 16 cores: bound the run to about two minutes
        args.steps = 3 if args.steps is None else min(args.steps, 40)
        args.warmup = 1 if args.warmup is None else min(args.warmup, 5)
        run_reference(args)
    else:
        args.steps = 2000 if args.steps is None else args.steps
        args.warmup = 20 if args.warmup is None else max(args.warmup, 3)
        if args.config == "demote_under_load":
            run_d5(args)
        else:
            run_gpu(args)


if __name__ == "__main__":
    main()
