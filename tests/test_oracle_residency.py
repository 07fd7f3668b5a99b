"""Pins of the page life-cycle oracle: the ordering rules of Sec. 3.1 / 3.3 as cases, and Eq. 3's released
bytes with the hand-computed size table.  CPU only."""
import os

import pytest


@pytest.fixture(scope="module")
def res():
    from oracle import residency
    return residency


def size_table():
    path = os.path.join(os.path.dirname(__file__), "golden", "page_bytes.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    return {int(r[2]): int(r[3]) for r in rows}


def test_offload_lowers_the_committed_bitwidth_first(res):
    M = size_table()
    row = res.Row(M)
    row.add_gpu_page(16, b"sixteen")
    row.commit(16)
    with pytest.raises(res.IllegalTransition):
        row.offload(16)                               # the committed page cannot leave
    row.add_gpu_page(4, b"four")                      # the demoted page
    assert row.gpu_bytes() == M[16] + M[4]
    row.commit(4)                                     # lower q_i first ...
    row.offload(16)                                   # ... then move the unneeded page
    assert row.state[16] == res.IN_TRANSFER and row.gpu_bytes() == M[16] + M[4]
    with pytest.raises(res.IllegalTransition):
        row.commit(16)
    row.transfer_done(16)
    assert row.state[16] == res.CPU
    # Eq. 3: going from 16 to 4 bits released M^16 - M^4 = 117440512 - 31195136 bytes
    assert M[16] - row.gpu_bytes() == 117440512 - 31195136 == 86245376


def test_reload_restores_the_page_before_the_commit(res):
    M = size_table()
    row = res.Row(M)
    row.add_gpu_page(16, b"sixteen")
    row.add_gpu_page(4, b"four")
    row.commit(4)
    row.offload(16)
    with pytest.raises(res.IllegalTransition):
        row.reload(16)                                # still on its way out
    row.transfer_done(16)
    with pytest.raises(res.IllegalTransition):
        row.commit(16)                                # CPU-resident
    with pytest.raises(res.IllegalTransition):
        row.offload(16)
    row.reload(16)
    with pytest.raises(res.IllegalTransition):
        row.commit(16)                                # in transfer: q_i is not raised yet
    assert row.committed == 4
    row.transfer_done(16)
    row.commit(16)
    assert row.committed == 16 and row.data[16] == b"sixteen"
    with pytest.raises(res.IllegalTransition):
        row.transfer_done(16)
    with pytest.raises(res.IllegalTransition):
        row.commit(8)                                 # no page at that bitwidth


def test_two_step_descent_releases_the_sum_of_the_steps(res):
    M = size_table()
    row = res.Row(M)
    row.add_gpu_page(16)
    row.commit(16)
    start = row.gpu_bytes()
    for lower, upper in ((4, 16), (2, 4)):
        row.add_gpu_page(lower)
        row.commit(lower)
        row.offload(upper)
        row.transfer_done(upper)
    assert start - row.gpu_bytes() == (M[16] - M[4]) + (M[4] - M[2]) == M[16] - M[2]
    assert sorted(b for b, s in row.state.items() if s == res.CPU) == [4, 16]


def test_planes_leave_above_the_committed_precision_and_return_before_it_is_raised(res):
    # a 14336 x 4096 block: a plane is one bit of every weight = 7,340,032 bytes; the leading planes with the
    # table states of the three bitwidths are 3584 tiles x 5632 bytes
    plane, top = 14336 * 4096 // 8, (14336 // 128) * (4096 // 128) * 5632
    assert (plane, top) == (7340032, 20185088)
    M = size_table()
    row = res.PlaneRow(top, plane)
    row.commit(4)
    for p in (3, 4):
        with pytest.raises(res.IllegalTransition):
            row.offload(p)                            # q_i = 4 reads both planes
    row.commit(3)                                     # lower q_i first ...
    with pytest.raises(res.IllegalTransition):
        row.offload(3)
    row.offload(4)                                    # ... then the plane it no longer reads moves out
    with pytest.raises(res.IllegalTransition):
        row.commit(4)                                 # on its way out
    assert row.gpu_bytes() == top + 2 * plane         # its buffer still exists
    row.transfer_done(4)
    assert row.gpu_bytes() == top + plane
    row.commit(2)
    row.offload(3)
    row.transfer_done(3)
    # Eq. 3 on the size table: 4 -> 2 bits releases M^4 - M^2 = two planes (the table state is the same size)
    assert 2 * plane == M[4] - M[2] == 31195136 - 16515072
    with pytest.raises(res.IllegalTransition):
        row.commit(3)                                 # CPU-resident
    with pytest.raises(res.IllegalTransition):
        row.transfer_done(3)                          # no transfer in flight
    row.reload(3)
    with pytest.raises(res.IllegalTransition):
        row.commit(3)                                 # still in transfer
    row.transfer_done(3)
    row.commit(3)
    with pytest.raises(res.IllegalTransition):
        row.commit(4)                                 # plane 4 is still away
    row.reload(4)
    row.transfer_done(4)
    row.commit(4)
    assert row.committed == 4 and row.gpu_bytes() == top + 2 * plane
    with pytest.raises(res.IllegalTransition):
        row.commit(5)
