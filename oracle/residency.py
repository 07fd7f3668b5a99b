"""Oracle of the page life-cycle: residency states, offload and reload of weight pages.  TEST INFRASTRUCTURE ONLY.

A plain state machine written from the rules of Sec. 3.1 and Sec. 3.3 (asynchronous page movement):

* every page of a page-table row is GPU-resident, CPU-resident or in transfer;
* offload: the committed bitwidth q_i is lowered FIRST, then the pages that are no longer needed move from
  GPU memory to CPU memory -- so the page a row is committed to can never be offloaded;
* reload: the page moves back to GPU memory FIRST; q_i is raised only once its state is GPU-resident;
* GPU memory released by going from bitwidth b to b' is M^b - M^b' (Eq. 3).

A row of ordinary pages has one page per bitwidth (group-wise codes), so "the pages above the committed
precision" are the pages of the row at higher bitwidths (class Row).  A row that holds a block of overlaid
bit-planes (Sec. 2.2) is the paper's own case: the unit of movement is a plane, plane p (3 or 4) is what reading
at p bits adds to reading at p - 1 bits, and the same two rules apply to planes (class PlaneRow).  Moving bytes
is the identity: what went out and came back holds the same bytes.

Only the tests import this module; it shares nothing with the CUDA sources.
"""
from __future__ import annotations

from typing import Dict, Optional

GPU, CPU, IN_TRANSFER, NONE = 0, 1, 2, 3


class IllegalTransition(Exception):
    pass


class Row:
    """The pages of one page-table row, keyed by bitwidth."""

    def __init__(self, page_bytes: Dict[int, int]):
        self.page_bytes = dict(page_bytes)          # size table M^b of the row
        self.state: Dict[int, int] = {}
        self.heading: Dict[int, int] = {}           # state a page in transfer will reach
        self.data: Dict[int, bytes] = {}            # the page's bytes, wherever they are
        self.committed: Optional[int] = None        # q_i

    def _st(self, bits: int) -> int:
        return self.state.get(bits, NONE)

    def add_gpu_page(self, bits: int, data: bytes = b""):
        if self._st(bits) in (CPU, IN_TRANSFER):
            raise IllegalTransition("a page of this bitwidth is away or on its way")
        self.state[bits] = GPU
        self.data[bits] = data

    def commit(self, bits: int):
        if self._st(bits) != GPU:
            raise IllegalTransition("q_i is only set to a bitwidth whose page is GPU-resident")
        self.committed = bits

    def offload(self, bits: int):
        if self._st(bits) != GPU:
            raise IllegalTransition("only a GPU-resident page can be offloaded")
        if self.committed == bits:
            raise IllegalTransition("lower q_i before moving the page out")
        self.state[bits] = IN_TRANSFER
        self.heading[bits] = CPU

    def reload(self, bits: int):
        if self._st(bits) != CPU:
            raise IllegalTransition("only a CPU-resident page can be reloaded")
        self.state[bits] = IN_TRANSFER
        self.heading[bits] = GPU

    def transfer_done(self, bits: int):
        if self._st(bits) != IN_TRANSFER:
            raise IllegalTransition("no transfer in flight")
        self.state[bits] = self.heading.pop(bits)

    def gpu_bytes(self) -> int:
        """GPU memory the row holds: resident pages, and pages in transfer (their buffers exist on both sides)."""
        return sum(self.page_bytes[b] for b, s in self.state.items() if s in (GPU, IN_TRANSFER))


class PlaneRow:
    """A page-table row that holds a block of overlaid bit-planes: the leading planes (the view at 2 bits, with the
    table state of every bitwidth) never leave the GPU; plane 3 and plane 4 are the third and the fourth bit of
    every code.  Read at q bits the row needs the planes 3 .. q."""

    def __init__(self, top_bytes: int, plane_bytes: int):
        self.top_bytes, self.plane_bytes = top_bytes, plane_bytes
        self.state: Dict[int, int] = {3: GPU, 4: GPU}
        self.heading: Dict[int, int] = {}
        self.committed: Optional[int] = None        # q_i

    def commit(self, q: int):
        if q not in (2, 3, 4):
            raise IllegalTransition("a block of bit-planes is read at 2, 3 or 4 bits")
        if any(self.state[p] != GPU for p in range(3, q + 1)):
            raise IllegalTransition("q_i is only raised once the planes it reads are GPU-resident")
        self.committed = q

    def offload(self, plane: int):
        if self.state.get(plane, NONE) != GPU:
            raise IllegalTransition("only a GPU-resident plane can be offloaded")
        if self.committed is not None and self.committed >= plane:
            raise IllegalTransition("lower q_i before moving a plane out that it reads")
        self.state[plane] = IN_TRANSFER
        self.heading[plane] = CPU

    def reload(self, plane: int):
        if self.state.get(plane, NONE) != CPU:
            raise IllegalTransition("only a CPU-resident plane can be reloaded")
        self.state[plane] = IN_TRANSFER
        self.heading[plane] = GPU

    def transfer_done(self, plane: int):
        if self.state.get(plane, NONE) != IN_TRANSFER:
            raise IllegalTransition("no transfer in flight")
        self.state[plane] = self.heading.pop(plane)

    def gpu_bytes(self) -> int:
        """GPU memory the row holds: the leading planes, and every further plane that is resident or in transfer."""
        return self.top_bytes + sum(self.plane_bytes for s in self.state.values() if s in (GPU, IN_TRANSFER))
