"""Thin ctypes binding of the C ABI declared in ``include/pw.h``.

Argument marshalling only: every step of the hot path runs inside ``libpw.so``.
PyTorch supplies device memory (``tensor.data_ptr()``) and streams.  There is no
CPU fallback: if the library cannot be loaded, importing names from here raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpw.so")

PW_OK = 0
STATUS_NAMES = {0: "PW_OK", 1: "PW_ERR_INVALID_ARG", 2: "PW_ERR_SHAPE", 3: "PW_ERR_BITS", 4: "PW_ERR_ALIGN",
                5: "PW_ERR_STATE", 6: "PW_ERR_NOMEM", 7: "PW_ERR_CUDA", 8: "PW_ERR_TIMEOUT"}
PW_GATE, PW_UP, PW_DOWN = 0, 1, 2
PW_MODE_AUTO, PW_MODE_SIMT, PW_MODE_TENSOR = 0, 1, 2
PW_LAYOUT_CANONICAL, PW_LAYOUT_TILED, PW_LAYOUT_PLANES = 0, 1, 2
PW_STATE_GPU_RESIDENT, PW_STATE_CPU_RESIDENT, PW_STATE_IN_TRANSFER, PW_STATE_NONE = 0, 1, 2, 3
GROUP = 128

# every symbol include/pw.h declares
EXPORTS = ("pw_workspace_bytes", "pw_create", "pw_destroy", "pw_page_bytes", "pw_quantize_block", "pw_demote_block",
           "pw_export_page", "pw_import_page", "pw_plane_bytes", "pw_quantize_planes", "pw_export_planes", "pw_set_page_table", "pw_get_page_table", "pw_query_row",
           "pw_offload_page", "pw_reload_page", "pw_page_state", "pw_drop_page",
           "pw_offload_plane", "pw_reload_plane", "pw_plane_state",
           "pw_moe_forward", "pw_moe_forward_host", "pw_get_routing", "pw_route_tokens_static", "pw_observe", "pw_observation_summary", "pw_plan_step", "pw_plan_queue_create", "pw_plan_queue_destroy", "pw_plan_queue_step", "pw_plan_queue_peek", "pw_kv_pressure_bytes",
           "pw_last_device_status",
           "pw_kernel_timing", "pw_get_kernel_times", "pw_launch_count", "pw_debug_set_wait", "pw_status_str")
KERNEL_NAMES = ("router", "permute", "gather", "ffn_gate_up", "ffn_down", "combine", "observe")
PW_OBS_FIELDS = 8
OBS_FIELD_NAMES = ("sum_r", "pairs", "sum_r_nx", "sum_r_nx2", "max_nx", "sum_r_nh", "sum_r_nh2", "max_nh")


class PwError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s" % (where, STATUS_NAMES.get(status, str(status))))


class pw_config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_experts", C.c_int32), ("n_shared", C.c_int32), ("hidden", C.c_int32),
                ("ffn", C.c_int32), ("group", C.c_int32), ("max_tokens", C.c_int32), ("max_top_k", C.c_int32),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class pw_page(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("scales", C.c_void_p), ("zps", C.c_void_p), ("rows", C.c_uint32),
                ("cols", C.c_uint32), ("group", C.c_uint16), ("bits", C.c_uint8), ("layout", C.c_uint8)]


class pw_table_entry(C.Structure):
    _fields_ = [("layer", C.c_int32), ("expert", C.c_int32), ("kind", C.c_int32), ("page", pw_page),
                ("desired_bits", C.c_uint8), ("state", C.c_uint8)]


class pw_plan_tables(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_experts", C.c_int32), ("n_shared", C.c_int32),
                ("committed", C.c_void_p), ("supported", C.c_void_p), ("sensitivity", C.c_void_p),
                ("page_bytes", C.c_void_p), ("mass", C.c_void_p), ("phi", C.c_void_p), ("head_w", C.c_void_p),
                ("head_a", C.c_void_p), ("head_c", C.c_void_p), ("alpha", C.c_float), ("rho_min", C.c_float),
                ("rho_max", C.c_float), ("epsilon", C.c_float), ("n_buckets", C.c_int32), ("n_stages", C.c_int32),
                ("bucket_share", C.c_void_p), ("bucket_mu", C.c_void_p), ("stage_floor", C.c_void_p)]


class pw_plan_item(C.Structure):
    _fields_ = [("layer", C.c_int32), ("expert", C.c_int32), ("kind", C.c_int32), ("from_bits", C.c_uint8),
                ("to_bits", C.c_uint8), ("released_bytes", C.c_uint64), ("damage", C.c_double)]


_lib = None


def load():
    """Loads libpw.so (built by ``paper_2607_16184_b200.build``).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libpw.so is missing: run `python -m paper_2607_16184_b200.build` (there is no fallback path)")
    L = C.CDLL(LIB_PATH)
    vp, i32, u32, sz = C.c_void_p, C.c_int, C.c_uint32, C.c_size_t
    L.pw_workspace_bytes.restype = sz
    L.pw_workspace_bytes.argtypes = [C.POINTER(pw_config)]
    L.pw_create.restype = i32
    L.pw_create.argtypes = [C.POINTER(vp), C.POINTER(pw_config)]
    L.pw_destroy.restype = i32
    L.pw_destroy.argtypes = [vp]
    L.pw_page_bytes.restype = sz
    L.pw_page_bytes.argtypes = [u32, u32, i32, i32, C.POINTER(sz), C.POINTER(sz), C.POINTER(sz)]
    L.pw_quantize_block.restype = i32
    L.pw_quantize_block.argtypes = [vp, vp, u32, u32, i32, C.POINTER(pw_page), vp]
    L.pw_demote_block.restype = i32
    L.pw_demote_block.argtypes = [vp, C.POINTER(pw_page), i32, C.POINTER(pw_page), vp]
    L.pw_export_page.restype = i32
    L.pw_export_page.argtypes = [vp, C.POINTER(pw_page), C.POINTER(pw_page), vp]
    L.pw_import_page.restype = i32
    L.pw_import_page.argtypes = [vp, C.POINTER(pw_page), C.POINTER(pw_page), vp]
    L.pw_set_page_table.restype = i32
    L.pw_set_page_table.argtypes = [vp, C.POINTER(pw_table_entry), sz, vp, C.POINTER(C.c_uint64)]
    L.pw_get_page_table.restype = vp
    L.pw_get_page_table.argtypes = [vp]
    L.pw_query_row.restype = i32
    L.pw_query_row.argtypes = [vp, i32, i32, i32, C.POINTER(pw_table_entry)]
    L.pw_offload_page.restype = i32
    L.pw_offload_page.argtypes = [vp, i32, i32, i32, C.POINTER(pw_page), vp, vp]
    L.pw_reload_page.restype = i32
    L.pw_reload_page.argtypes = [vp, i32, i32, i32, i32, vp, C.POINTER(pw_page), vp]
    L.pw_page_state.restype = i32
    L.pw_page_state.argtypes = [vp, i32, i32, i32, i32, C.POINTER(C.c_int)]
    L.pw_drop_page.restype = i32
    L.pw_drop_page.argtypes = [vp, i32, i32, i32, i32]
    L.pw_offload_plane.restype = i32
    L.pw_offload_plane.argtypes = [vp, i32, i32, i32, C.POINTER(pw_page), i32, vp, vp]
    L.pw_reload_plane.restype = i32
    L.pw_reload_plane.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp]
    L.pw_plane_state.restype = i32
    L.pw_plane_state.argtypes = [vp, i32, i32, i32, i32, C.POINTER(C.c_int)]
    L.pw_moe_forward.restype = i32
    L.pw_moe_forward.argtypes = [vp, i32, vp, vp, i32, i32, vp, vp, i32, vp]
    L.pw_moe_forward_host.restype = i32
    L.pw_moe_forward_host.argtypes = [vp, i32, vp, vp, i32, i32, vp, i32, vp]
    L.pw_route_tokens_static.restype = i32
    L.pw_route_tokens_static.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp]
    L.pw_get_routing.restype = i32
    L.pw_get_routing.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.pw_observe.restype = i32
    L.pw_observe.argtypes = [vp, vp, vp]
    L.pw_observation_summary.restype = i32
    L.pw_observation_summary.argtypes = [vp, i32, vp, vp, vp]
    L.pw_plan_step.restype = i32
    L.pw_plan_step.argtypes = [C.POINTER(pw_plan_tables), C.c_uint64, C.POINTER(pw_plan_item), sz, C.POINTER(sz),
                               C.POINTER(C.c_uint64), C.POINTER(C.c_int32)]
    L.pw_kv_pressure_bytes.restype = C.c_uint64
    L.pw_kv_pressure_bytes.argtypes = [C.c_int64, C.c_int64, C.c_uint64]
    L.pw_last_device_status.restype = i32
    L.pw_last_device_status.argtypes = [vp]
    L.pw_kernel_timing.restype = i32
    L.pw_kernel_timing.argtypes = [vp, i32]
    L.pw_get_kernel_times.restype = i32
    L.pw_get_kernel_times.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_uint64)]
    L.pw_plane_bytes.restype = C.c_size_t
    L.pw_plane_bytes.argtypes = [C.c_uint32, C.c_uint32, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    L.pw_quantize_planes.restype = C.c_int
    L.pw_quantize_planes.argtypes = [vp, vp, C.c_uint32, C.c_uint32, C.POINTER(pw_page), vp]
    L.pw_export_planes.restype = C.c_int
    L.pw_export_planes.argtypes = [vp, C.POINTER(pw_page), C.POINTER(pw_page), vp]
    L.pw_plan_queue_create.restype = C.c_int
    L.pw_plan_queue_create.argtypes = [C.POINTER(C.c_void_p), C.c_int32]
    L.pw_plan_queue_destroy.restype = C.c_int
    L.pw_plan_queue_destroy.argtypes = [vp]
    L.pw_plan_queue_step.restype = C.c_int
    L.pw_plan_queue_step.argtypes = [vp, C.POINTER(pw_plan_tables), C.c_int64, C.c_int64, C.c_uint64, C.c_uint64,
                                     C.POINTER(pw_plan_item), C.c_size_t, C.POINTER(C.c_size_t), C.POINTER(C.c_uint64),
                                     C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    L.pw_plan_queue_peek.restype = C.c_int
    L.pw_plan_queue_peek.argtypes = [vp, C.c_int32, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64), C.POINTER(C.c_size_t),
                                     C.POINTER(C.c_uint64)]
    L.pw_launch_count.restype = C.c_uint64
    L.pw_launch_count.argtypes = [vp]
    L.pw_debug_set_wait.restype = C.c_int
    L.pw_debug_set_wait.argtypes = [vp, C.c_uint32, C.c_uint32]
    L.pw_status_str.restype = C.c_char_p
    L.pw_status_str.argtypes = [i32]
    _lib = L
    return L


def _check(st: int, where: str):
    if st != PW_OK:
        raise PwError(st, where)


def _stream_ptr(stream: Optional[torch.cuda.Stream]):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def pw_page_bytes(rows: int, cols: int, bits: int, group: int = GROUP) -> Tuple[int, int, int, int]:
    """(total, codes, scales, zps) bytes -- the size table M_i^b of Eq. 3.  total == 0 means invalid arguments."""
    a, b, c = C.c_size_t(), C.c_size_t(), C.c_size_t()
    tot = load().pw_page_bytes(rows, cols, bits, group, C.byref(a), C.byref(b), C.byref(c))
    return int(tot), int(a.value), int(b.value), int(c.value)


def pw_kv_pressure_bytes(free_block_threshold: int, free_blocks: int, kv_block_bytes: int) -> int:
    """Eq. 7: bytes the planner has to release."""
    return int(load().pw_kv_pressure_bytes(free_block_threshold, free_blocks, kv_block_bytes))


def _plan_tables(n_layers, n_experts, n_shared, committed, supported, sensitivity, page_bytes, mass, bucket_share,
                 bucket_mu, stage_floor, phi, heads, alpha, rho_min, rho_max, epsilon):
    """pw_plan_tables over host arrays (numpy; shapes as in include/pw.h) + the arrays it points into."""
    import numpy as np
    keep = []

    def ptr(a, dt):
        if a is None:
            return None
        a = np.ascontiguousarray(a, dt)
        keep.append(a)
        return a.ctypes.data

    floors = np.ascontiguousarray(stage_floor, np.uint8)
    t = pw_plan_tables()
    t.n_layers, t.n_experts, t.n_shared = n_layers, n_experts, n_shared
    t.committed, t.supported = ptr(committed, np.uint8), ptr(supported, np.uint8)
    t.sensitivity, t.page_bytes = ptr(sensitivity, np.float32), ptr(page_bytes, np.uint64)
    t.mass, t.phi = ptr(mass, np.float32), ptr(phi, np.float32)
    if heads is not None:
        t.head_w, t.head_a, t.head_c = ptr(heads["w"], np.float32), ptr(heads["a"], np.float32), ptr(heads["c"], np.float32)
    t.alpha, t.rho_min, t.rho_max, t.epsilon = alpha, rho_min, rho_max, epsilon
    t.n_buckets, t.n_stages = floors.shape[1], floors.shape[0]
    t.bucket_share, t.bucket_mu, t.stage_floor = ptr(bucket_share, np.float32), ptr(bucket_mu, np.float32), ptr(floors, np.uint8)
    return t, keep


def _plan_items(items, n):
    return [(it.layer, it.expert, it.kind, it.from_bits, it.to_bits, it.damage) for it in items[:n]]


def pw_plan_step(n_layers: int, n_experts: int, n_shared: int, committed, supported, sensitivity, page_bytes, mass,
                 bucket_share, bucket_mu, stage_floor, target: int, phi=None, heads=None, alpha: float = 1.0,
                 rho_min: float = -1.0, rho_max: float = 1.0, epsilon: float = 1e-9):
    """One planner step on host arrays (numpy; shapes as in include/pw.h).  Returns (steps, released bytes,
    stage) with steps as tuples (layer, expert, kind, from_bits, to_bits, damage)."""
    t, keep = _plan_tables(n_layers, n_experts, n_shared, committed, supported, sensitivity, page_bytes, mass, bucket_share,
                           bucket_mu, stage_floor, phi, heads, alpha, rho_min, rho_max, epsilon)
    cap = n_layers * (n_experts + n_shared) * 3 * 4
    items = (pw_plan_item * cap)()
    n, rel, stage = C.c_size_t(), C.c_uint64(), C.c_int32()
    _check(load().pw_plan_step(C.byref(t), target, items, cap, C.byref(n), C.byref(rel), C.byref(stage)), "pw_plan_step")
    return _plan_items(items, n.value), int(rel.value), int(stage.value)


class PlanQueue:
    """The plan queue of Alg. 1 (host code): ``step`` is one PlanStep -- refresh every stage's candidate plan from
    the tables, hand out a plan only under KV-cache pressure."""

    def __init__(self, n_stages: int):
        self.handle = C.c_void_p()
        _check(load().pw_plan_queue_create(C.byref(self.handle), n_stages), "pw_plan_queue_create")

    def close(self):
        if self.handle:
            load().pw_plan_queue_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def step(self, n_layers, n_experts, n_shared, committed, supported, sensitivity, page_bytes, mass, bucket_share,
             bucket_mu, stage_floor, free_block_threshold: int, free_blocks: int, kv_block_bytes: int,
             lookahead_bytes: int, phi=None, heads=None, alpha: float = 1.0, rho_min: float = -1.0, rho_max: float = 1.0,
             epsilon: float = 1e-9):
        """Returns (triggered, steps, released bytes, stage); without pressure: (False, [], 0, -1)."""
        t, keep = _plan_tables(n_layers, n_experts, n_shared, committed, supported, sensitivity, page_bytes, mass,
                               bucket_share, bucket_mu, stage_floor, phi, heads, alpha, rho_min, rho_max, epsilon)
        cap = n_layers * (n_experts + n_shared) * 3 * 4
        items = (pw_plan_item * cap)()
        n, rel, stage, trig = C.c_size_t(), C.c_uint64(), C.c_int32(), C.c_int32()
        _check(load().pw_plan_queue_step(self.handle, C.byref(t), free_block_threshold, free_blocks, kv_block_bytes,
                                         lookahead_bytes, items, cap, C.byref(n), C.byref(rel), C.byref(stage),
                                         C.byref(trig)), "pw_plan_queue_step")
        return bool(trig.value), _plan_items(items, n.value), int(rel.value), int(stage.value)

    def peek(self, stage: int):
        """(target, released bytes, number of steps, refreshed at planner step) of a stage's queued candidate."""
        tg, rel, n, at = C.c_uint64(), C.c_uint64(), C.c_size_t(), C.c_uint64()
        _check(load().pw_plan_queue_peek(self.handle, stage, C.byref(tg), C.byref(rel), C.byref(n), C.byref(at)),
               "pw_plan_queue_peek")
        return int(tg.value), int(rel.value), int(n.value), int(at.value)


def pw_route_tokens_static(router_logits: torch.Tensor, top_k: int,
                           stream: Optional[torch.cuda.Stream] = None) -> Dict[str, torch.Tensor]:
    """Router + stable grouping without a context or workspace (for callers that must not allocate
    device memory inside the call; the output tensors here are made by the caller's allocator, torch)."""
    assert router_logits.dtype == torch.float32 and router_logits.is_contiguous() and router_logits.is_cuda
    T, E = router_logits.shape
    d = router_logits.device
    r = {"topk_ids": torch.empty(T, top_k, dtype=torch.int32, device=d),
         "gates": torch.empty(T, top_k, dtype=torch.float32, device=d),
         "counts": torch.empty(E, dtype=torch.int32, device=d),
         "offsets": torch.empty(E + 1, dtype=torch.int32, device=d),
         "perm": torch.empty(T * top_k, dtype=torch.int32, device=d)}
    with torch.cuda.device(d):
        _check(load().pw_route_tokens_static(router_logits.data_ptr(), T, E, top_k, r["topk_ids"].data_ptr(),
                                             r["gates"].data_ptr(), r["counts"].data_ptr(), r["offsets"].data_ptr(),
                                             r["perm"].data_ptr(), _stream_ptr(stream)), "pw_route_tokens_static")
    return r


class Page:
    """Device buffers of one weight page plus its ``pw_page`` header.

    A TILED page is one buffer (``codes``) of the total page size; a CANONICAL page below 16 bits has
    separate ``codes``, ``scales`` and ``zps`` buffers.
    """

    def __init__(self, rows: int, cols: int, bits: int, device="cuda", layout: int = PW_LAYOUT_TILED):
        tot, cb, sb, zb = pw_page_bytes(rows, cols, bits)
        if tot == 0:
            # unallocatable request: keep a header with null buffers so the C call reports the precise error
            self.codes = self.scales = self.zps = None
            self.c = pw_page(None, None, None, rows, cols, GROUP, bits & 0xff, layout)
            self.nbytes = 0
            return
        if layout == PW_LAYOUT_TILED:
            cb, sb, zb = tot, 0, 0
        self.codes = torch.empty(cb, dtype=torch.uint8, device=device)
        self.scales = torch.empty(sb // 2, dtype=torch.float16, device=device) if sb else None
        self.zps = torch.empty(zb // 2, dtype=torch.float16, device=device) if zb else None
        self.c = pw_page(self.codes.data_ptr(), self.scales.data_ptr() if sb else None,
                         self.zps.data_ptr() if zb else None, rows, cols, GROUP, bits, layout)
        self.nbytes = tot

    rows = property(lambda self: self.c.rows)
    cols = property(lambda self: self.c.cols)
    bits = property(lambda self: self.c.bits)
    layout = property(lambda self: self.c.layout)


def pw_plane_bytes(rows: int, cols: int) -> Tuple[int, int, int]:
    """(total, TOP buffer, one bit-plane buffer) bytes of a bit-plane block."""
    t, b = C.c_size_t(), C.c_size_t()
    tot = load().pw_plane_bytes(rows, cols, C.byref(t), C.byref(b))
    return int(tot), int(t.value), int(b.value)


class PlanePage:
    """A bit-plane block (three device buffers) read at ``bits`` in {2, 3, 4}: the ``pw_page`` header of layout
    PW_LAYOUT_PLANES.  ``at(q)`` gives the same buffers at another bitwidth -- lowering or raising the precision
    is a new header, nothing else; with ``detach=True`` the header no longer names the planes q does not need."""

    def __init__(self, rows: int, cols: int, device="cuda", _buffers=None, bits: int = 4, detach: bool = False):
        if _buffers is None:
            _, tb, bb = pw_plane_bytes(rows, cols)
            _buffers = (torch.empty(tb, dtype=torch.uint8, device=device), torch.empty(bb, dtype=torch.uint8, device=device),
                        torch.empty(bb, dtype=torch.uint8, device=device))
        self.top, self.bit1, self.bit0 = _buffers
        self.codes = self.top
        p1 = self.bit1.data_ptr() if (bits >= 3 or not detach) else None
        p0 = self.bit0.data_ptr() if (bits == 4 or not detach) else None
        self.c = pw_page(self.top.data_ptr(), p1, p0, rows, cols, GROUP, bits, PW_LAYOUT_PLANES)
        self.nbytes = pw_page_bytes(rows, cols, bits)[0] if bits in (2, 3, 4) else 0

    rows = property(lambda self: self.c.rows)
    cols = property(lambda self: self.c.cols)
    bits = property(lambda self: self.c.bits)
    layout = property(lambda self: self.c.layout)

    def at(self, bits: int, detach: bool = False) -> "PlanePage":
        return PlanePage(self.rows, self.cols, _buffers=(self.top, self.bit1, self.bit0), bits=bits, detach=detach)


class Context:
    """Owns the workspace tensor and the ``pw_ctx``; methods carry the names of the C calls."""

    GUARD_BYTE = 0xA5

    def __init__(self, n_layers: int, n_experts: int, n_shared: int, hidden: int, ffn: int, max_tokens: int,
                 max_top_k: int, device="cuda", guard_bytes: int = 0):
        """``guard_bytes`` > 0 puts that many bytes of a known pattern in front of and behind the workspace
        (``workspace_guards_intact`` looks at them): a check that no kernel writes outside it."""
        self.L = load()
        self.device = torch.device(device)
        cfg = pw_config(n_layers, n_experts, n_shared, hidden, ffn, GROUP, max_tokens, max_top_k, None, 0)
        nbytes = self.L.pw_workspace_bytes(C.byref(cfg))
        if nbytes == 0:
            raise PwError(1, "pw_workspace_bytes")
        guard = (guard_bytes + 255) // 256 * 256
        self.workspace = torch.full((nbytes + 256 + 2 * guard,), self.GUARD_BYTE, dtype=torch.uint8, device=self.device) \
            if guard else torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + guard + 255) // 256 * 256
        self._ws_span = (base - self.workspace.data_ptr(), nbytes)
        cfg.workspace, cfg.workspace_bytes = base, nbytes
        self.cfg = cfg
        self.handle = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(self.L.pw_create(C.byref(self.handle), C.byref(cfg)), "pw_create")
        self.n_segments = n_experts + n_shared
        self._committed = {}          # (layer, expert, kind) -> the page the row points to
        self.obs = None               # accumulators of the observation taps while they are on

    def workspace_guards_intact(self) -> bool:
        """True when the bytes in front of and behind the workspace still hold the guard pattern."""
        off, nbytes = self._ws_span
        torch.cuda.synchronize(self.device)
        front, back = self.workspace[:off], self.workspace[off + nbytes:]
        return bool((front == self.GUARD_BYTE).all().item()) and bool((back == self.GUARD_BYTE).all().item())

    def close(self):
        if self.handle:
            self.L.pw_destroy(self.handle)      # waits for the device: nothing reads the pages any more
            self.handle = C.c_void_p()
            self._committed = {}
            self.obs = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- pages ----
    def pw_quantize_block(self, w_fp16: torch.Tensor, bits: int, dst: Optional[Page] = None,
                          stream: Optional[torch.cuda.Stream] = None) -> Page:
        assert w_fp16.dtype == torch.float16 and w_fp16.is_contiguous() and w_fp16.is_cuda
        rows, cols = w_fp16.shape
        dst = dst or Page(rows, cols, bits, self.device)
        _check(self.L.pw_quantize_block(self.handle, w_fp16.data_ptr(), rows, cols, bits, C.byref(dst.c),
                                        _stream_ptr(stream)), "pw_quantize_block")
        return dst

    def pw_demote_block(self, src: Page, dst_bits: int, dst: Optional[Page] = None,
                        stream: Optional[torch.cuda.Stream] = None) -> Page:
        dst = dst or Page(src.rows, src.cols, dst_bits, self.device)
        _check(self.L.pw_demote_block(self.handle, C.byref(src.c), dst_bits, C.byref(dst.c), _stream_ptr(stream)),
               "pw_demote_block")
        return dst

    def pw_export_page(self, src: Page, stream: Optional[torch.cuda.Stream] = None) -> Page:
        dst = Page(src.rows, src.cols, src.bits, self.device, PW_LAYOUT_CANONICAL)
        _check(self.L.pw_export_page(self.handle, C.byref(src.c), C.byref(dst.c), _stream_ptr(stream)),
               "pw_export_page")
        return dst

    def pw_quantize_planes(self, w_fp16: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> PlanePage:
        assert w_fp16.dtype == torch.float16 and w_fp16.is_contiguous() and w_fp16.is_cuda
        rows, cols = w_fp16.shape
        dst = PlanePage(rows, cols, self.device)
        _check(self.L.pw_quantize_planes(self.handle, w_fp16.data_ptr(), rows, cols, C.byref(dst.c), _stream_ptr(stream)),
               "pw_quantize_planes")
        return dst

    def pw_export_planes(self, src: PlanePage, stream: Optional[torch.cuda.Stream] = None) -> Page:
        dst = Page(src.rows, src.cols, src.bits, self.device, PW_LAYOUT_CANONICAL)
        _check(self.L.pw_export_planes(self.handle, C.byref(src.c), C.byref(dst.c), _stream_ptr(stream)),
               "pw_export_planes")
        return dst

    def pw_import_page(self, src: Page, stream: Optional[torch.cuda.Stream] = None) -> Page:
        dst = Page(src.rows, src.cols, src.bits, self.device, PW_LAYOUT_TILED)
        _check(self.L.pw_import_page(self.handle, C.byref(src.c), C.byref(dst.c), _stream_ptr(stream)),
               "pw_import_page")
        return dst

    # ---- page table ----
    def pw_set_page_table(self, entries: Sequence[Tuple[int, int, int, Page]],
                          stream: Optional[torch.cuda.Stream] = None, desired_bits: int = 0,
                          state: int = PW_STATE_GPU_RESIDENT) -> int:
        """entries: (layer, expert, kind, page).  Returns the table epoch after the commit."""
        arr = (pw_table_entry * len(entries))()
        for i, (layer, expert, kind, page) in enumerate(entries):
            arr[i].layer, arr[i].expert, arr[i].kind = layer, expert, kind
            arr[i].page = page.c
            arr[i].desired_bits = desired_bits
            arr[i].state = state
        epoch = C.c_uint64()
        _check(self.L.pw_set_page_table(self.handle, arr, len(entries), _stream_ptr(stream), C.byref(epoch)),
               "pw_set_page_table")
        # the library only borrows page buffers: keep every committed page alive until its row is replaced
        for layer, expert, kind, page in entries:
            self._committed[(layer, expert, kind)] = page
        return int(epoch.value)

    def pw_query_row(self, layer: int, expert: int, kind: int) -> pw_table_entry:
        out = pw_table_entry()
        _check(self.L.pw_query_row(self.handle, layer, expert, kind, C.byref(out)), "pw_query_row")
        return out

    # ---- residency ----
    def pw_offload_page(self, layer: int, expert: int, kind: int, page: Page,
                        stream: Optional[torch.cuda.Stream] = None, host: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Starts the copy of a (not committed) page to pinned host memory; returns the host buffer."""
        nbytes = pw_page_bytes(page.rows, page.cols, page.bits)[0]
        if host is None:
            host = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
        assert host.numel() >= nbytes and not host.is_cuda
        _check(self.L.pw_offload_page(self.handle, layer, expert, kind, C.byref(page.c), host.data_ptr(),
                                      _stream_ptr(stream)), "pw_offload_page")
        return host

    def pw_reload_page(self, layer: int, expert: int, kind: int, bits: int, host: torch.Tensor,
                       stream: Optional[torch.cuda.Stream] = None) -> Page:
        """Starts the copy of an offloaded page back into a fresh device buffer; returns the page."""
        rows, cols = (self.cfg.hidden, self.cfg.ffn) if kind == PW_DOWN else (self.cfg.ffn, self.cfg.hidden)
        dst = Page(rows, cols, bits, self.device)
        _check(self.L.pw_reload_page(self.handle, layer, expert, kind, bits, host.data_ptr(), C.byref(dst.c),
                                     _stream_ptr(stream)), "pw_reload_page")
        return dst

    def pw_page_state(self, layer: int, expert: int, kind: int, bits: int) -> int:
        st = C.c_int()
        _check(self.L.pw_page_state(self.handle, layer, expert, kind, bits, C.byref(st)), "pw_page_state")
        return int(st.value)

    def pw_drop_page(self, layer: int, expert: int, kind: int, bits: int):
        _check(self.L.pw_drop_page(self.handle, layer, expert, kind, bits), "pw_drop_page")

    def pw_offload_plane(self, layer: int, expert: int, kind: int, block: "PlanePage", plane: int,
                         stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """Starts the copy of plane 3 (BIT1) or 4 (BIT0) of a bit-plane block to pinned host memory; returns it."""
        _, _, bb = pw_plane_bytes(block.rows, block.cols)
        host = torch.empty(bb, dtype=torch.uint8).pin_memory()
        _check(self.L.pw_offload_plane(self.handle, layer, expert, kind, C.byref(block.c), plane, host.data_ptr(),
                                       _stream_ptr(stream)), "pw_offload_plane")
        return host

    def pw_reload_plane(self, layer: int, expert: int, kind: int, plane: int, host: torch.Tensor,
                        stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """Starts the copy of an offloaded plane back into a fresh device buffer; returns the buffer."""
        dst = torch.empty(host.numel(), dtype=torch.uint8, device=self.device)
        _check(self.L.pw_reload_plane(self.handle, layer, expert, kind, plane, host.data_ptr(), dst.data_ptr(),
                                      _stream_ptr(stream)), "pw_reload_plane")
        return dst

    def pw_plane_state(self, layer: int, expert: int, kind: int, plane: int) -> int:
        st = C.c_int()
        _check(self.L.pw_plane_state(self.handle, layer, expert, kind, plane, C.byref(st)), "pw_plane_state")
        return int(st.value)

    # ---- forward ----
    def pw_moe_forward(self, layer: int, hidden: torch.Tensor, router_logits: torch.Tensor, top_k: int,
                       out: Optional[torch.Tensor] = None, mode: int = PW_MODE_AUTO,
                       stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        assert hidden.dtype == torch.float16 and hidden.is_contiguous()
        assert router_logits.dtype == torch.float32 and router_logits.is_contiguous()
        T, H = hidden.shape
        if out is None:
            out = torch.empty(T, H, dtype=torch.float32, device=hidden.device)
        table = self.L.pw_get_page_table(self.handle)
        _check(self.L.pw_moe_forward(self.handle, layer, hidden.data_ptr(), router_logits.data_ptr(), T, top_k,
                                     table, out.data_ptr(), mode, _stream_ptr(stream)), "pw_moe_forward")
        return out

    def pw_moe_forward_host(self, layer: int, hidden_host: torch.Tensor, logits_host: torch.Tensor, top_k: int,
                            out_host: torch.Tensor, mode: int = PW_MODE_AUTO,
                            stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """Host-buffer variant: the three tensors are (preferably pinned) CPU tensors."""
        assert not hidden_host.is_cuda and not logits_host.is_cuda and not out_host.is_cuda
        assert hidden_host.dtype == torch.float16 and logits_host.dtype == torch.float32
        assert out_host.dtype == torch.float32 and out_host.is_contiguous()
        T = hidden_host.shape[0]
        _check(self.L.pw_moe_forward_host(self.handle, layer, hidden_host.data_ptr(), logits_host.data_ptr(), T,
                                          top_k, out_host.data_ptr(), mode, _stream_ptr(stream)),
               "pw_moe_forward_host")
        return out_host

    def pw_get_routing(self, T: int, top_k: int, stream: Optional[torch.cuda.Stream] = None) -> Dict[str, torch.Tensor]:
        E = self.cfg.n_experts
        d = self.device
        r = {"topk_ids": torch.empty(T, top_k, dtype=torch.int32, device=d),
             "gates": torch.empty(T, top_k, dtype=torch.float32, device=d),
             "counts": torch.empty(E, dtype=torch.int32, device=d),
             "offsets": torch.empty(E + 1, dtype=torch.int32, device=d),
             "perm": torch.empty(T * top_k, dtype=torch.int32, device=d)}
        _check(self.L.pw_get_routing(self.handle, r["topk_ids"].data_ptr(), r["gates"].data_ptr(),
                                     r["counts"].data_ptr(), r["offsets"].data_ptr(), r["perm"].data_ptr(),
                                     _stream_ptr(stream)), "pw_get_routing")
        return r

    def pw_observe(self, enable: bool = True, stream: Optional[torch.cuda.Stream] = None) -> Optional[torch.Tensor]:
        """Switches the observation taps on (fresh, zeroed accumulators [n_layers, S, 8]) or off."""
        if not enable:
            _check(self.L.pw_observe(self.handle, None, _stream_ptr(stream)), "pw_observe")
            self.obs = None
            return None
        S = self.cfg.n_experts + self.cfg.n_shared
        self.obs = torch.empty(self.cfg.n_layers, S, PW_OBS_FIELDS, dtype=torch.float32, device=self.device)
        _check(self.L.pw_observe(self.handle, self.obs.data_ptr(), _stream_ptr(stream)), "pw_observe")
        return self.obs

    def pw_observation_summary(self, layer: int, stream: Optional[torch.cuda.Stream] = None):
        """(mass [E], phi [S, 3, 3]) of one layer, computed on the device from the accumulators."""
        S = self.cfg.n_experts + self.cfg.n_shared
        mass = torch.empty(self.cfg.n_experts, dtype=torch.float32, device=self.device)
        phi = torch.empty(S, 3, 3, dtype=torch.float32, device=self.device)
        _check(self.L.pw_observation_summary(self.handle, layer, mass.data_ptr(), phi.data_ptr(),
                                             _stream_ptr(stream)), "pw_observation_summary")
        return mass, phi

    def pw_last_device_status(self) -> int:
        return int(self.L.pw_last_device_status(self.handle))

    def pw_kernel_timing(self, enable: bool):
        _check(self.L.pw_kernel_timing(self.handle, 1 if enable else 0), "pw_kernel_timing")

    def pw_get_kernel_times(self):
        """({kernel name: summed ms}, forward calls covered) since timing was last enabled."""
        ms = (C.c_double * len(KERNEL_NAMES))()
        calls = C.c_uint64()
        _check(self.L.pw_get_kernel_times(self.handle, ms, C.byref(calls)), "pw_get_kernel_times")
        return {n: float(ms[i]) for i, n in enumerate(KERNEL_NAMES)}, int(calls.value)

    def pw_launch_count(self) -> int:
        return int(self.L.pw_launch_count(self.handle))

    def pw_debug_set_wait(self, polls: int = 0, hook: int = 0) -> None:
        """Wait limit of the gate/up FFN kernel (0 = the default 2 s, else the 4 ms test build) and test hooks."""
        _check(self.L.pw_debug_set_wait(self.handle, polls, hook), "pw_debug_set_wait")
