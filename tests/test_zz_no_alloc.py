"""bls_route_table_rr_static: the router for callers that cannot allocate device
memory (a process whose GPU memory belongs to another framework's pool, a plugin
with fixed buffers).  Its scratch is a static device array shared by all calls
and keeps the previous call's contents, so every case calls it at least twice in
a row with different inputs.  Every output is compared bit for bit with the CPU
oracle's routing artefacts, and also with the plan-based router (bls_route +
bls_view).  This file is collected last on purpose.  GPU only."""
import ctypes as C

import numpy as np
import pytest
import torch

import bls_inputs as bi
import oracle
import paper_2512_19342_b200 as bls
from test_gpu_parity import check_route

pytestmark = pytest.mark.gpu


class Buffers:
    """The caller's buffers of the static entry point, allocated once up front."""

    def __init__(self, w, cap):
        P, T, b = w.P, w.T, w.local_batch
        self.rows = torch.tensor([t.rows for t in w.tables], dtype=torch.int64, device="cuda")
        self.sendcounts = torch.empty(P, P, dtype=torch.int32, device="cuda")
        self.sdispls = torch.empty(P, P, dtype=torch.int32, device="cuda")
        self.sendbuf = torch.empty(P, cap, dtype=torch.int32, device="cuda")
        self.sub_start = torch.empty(P, T * b + 1, dtype=torch.int32, device="cuda")
        self.status = torch.empty(1, dtype=torch.int32, device="cuda")

    def route(self, w, ids, off):
        self.sendbuf.fill_(-7)
        bls.bls_route_table_rr_static(self.rows, w.P, w.local_batch, torch.from_numpy(ids).cuda(),
                                      torch.from_numpy(off).cuda(), self.sendcounts, self.sdispls, self.sendbuf,
                                      self.sub_start, self.status)
        torch.cuda.synchronize()

    def view(self):
        return {"sendcounts": self.sendcounts, "sdispls": self.sdispls, "sendbuf": self.sendbuf,
                "sub_start": self.sub_start, "sub_bag_major": False}


def capacity(w, inputs):
    tb = w.T * w.local_batch
    cap = max(int(np.diff(off[::tb].astype(np.int64)).max()) for _, off in inputs) + 13
    return (cap + 3) // 4 * 4


def check_against_oracle_and_plan(w, buf, ids, off, plan=None, it=0):
    """Static router's outputs of one call: vs the oracle (counts, displacements, packed
    buffers, sub-bag lengths), nothing written past a rank's total, and vs the plan router."""
    assert buf.status.item() == 0
    check_route(w, buf.view(), ids, off, recv_side=False)
    per_rank = np.diff(off[::w.T * w.local_batch].astype(np.int64))
    for src in range(w.P):
        assert torch.all(buf.sendbuf[src, int(per_rank[src]):] == -7)
    if plan is not None:
        d_ids, d_off = torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda()
        bls.bls_route(plan, it, d_ids, d_off)
        ref = bls.bls_view(plan, it)
        torch.cuda.synchronize()
        assert torch.equal(buf.sendcounts, ref["sendcounts"])
        assert torch.equal(buf.sdispls, ref["sdispls"])
        assert torch.equal(buf.sub_start, ref["sub_start"])
        for src in range(w.P):
            n = int(per_rank[src])
            assert torch.equal(buf.sendbuf[src, :n], ref["sendbuf"][src, :n]), (it, src)
        bls.bls_lookup(plan, it)


SHAPES = [
    ("cfg3_small", lambda: bi.workload(3, 0.02, 0.03)),                                     # 26 tables, P=8, b=61: one tile per table
    ("two_tiles_per_table", lambda: bi.tiny_workload(T=5, P=3, b=300, rows=400, dim=8, lengths="poisson10")),
    ("fewer_tables_than_ranks", lambda: bi.tiny_workload(T=3, P=8, b=40, rows=90, dim=8, lengths="mixed")),
]


@pytest.mark.parametrize("name,mk", SHAPES, ids=[s[0] for s in SHAPES])
def test_static_router_matches_oracle_twice_in_a_row(name, mk):
    w = mk()
    tabs = [torch.empty(t.rows, t.dim, device="cuda") for t in w.tables]   # values are not read by the router
    inputs = [bi.make_iteration(w, it) for it in (0, 1)]
    cap = capacity(w, inputs)
    plan = bls.bls_plan(tabs, "table_rr", w.P, w.local_batch, 0, cap)
    buf = Buffers(w, cap)
    for it, (ids, off) in enumerate(inputs):
        buf.route(w, ids, off)
        check_against_oracle_and_plan(w, buf, ids, off, plan, it)
    assert bls.bls_status(plan)[0] == bls.BLS_OK


def test_stale_scratch_of_a_larger_call_does_not_leak_into_a_smaller_one():
    """A call that uses much of the static array, then one that uses little of it, then the
    large one again: each sees only its own chunk bases."""
    big = bi.tiny_workload(T=70, P=16, b=9, rows=40, dim=8, lengths="mixed")          # P * (T + 1) = 1136 entries
    small = bi.tiny_workload(T=2, P=3, b=130, rows=50, dim=8, lengths="poisson10")    # 9 entries
    for w in (big, small, big, small):
        ids, off = bi.make_iteration(w, 1)
        buf = Buffers(w, capacity(w, [(ids, off)]))
        buf.route(w, ids, off)
        check_against_oracle_and_plan(w, buf, ids, off)


def test_static_router_reports_bad_input_in_its_status_word():
    """Out-of-range ID -> 4, send buffer too small -> 2, non-monotone offsets -> 1; nothing
    is written outside the caller's buffers and the device stays usable."""
    w = bi.tiny_workload(T=4, P=2, b=150, rows=30, dim=8, lengths="one")
    ids, off = bi.make_iteration(w, 0)
    cap = capacity(w, [(ids, off)])
    buf = Buffers(w, cap)
    bad = ids.copy()
    bad[7] = 30
    bad[401] = -1
    buf.route(w, bad, off)
    assert buf.status.item() == 4
    fixed = bad.copy()
    fixed[[7, 401]] = 0                                     # an out-of-range ID is replaced by row 0
    want = oracle.route(w.P, w.T, w.local_batch, "table_rr", [t.rows for t in w.tables], fixed, off)
    assert np.array_equal(buf.sendcounts.cpu().numpy(), want["sendcounts"])
    n0 = int(off[w.T * w.local_batch])
    assert np.array_equal(buf.sendbuf[0, :n0].cpu().numpy(), want["sendbuf"][:n0])
    # a send buffer of 64 entries per rank cannot hold 600: reported, and the guard words after it stay untouched
    guard = torch.full((w.P * 64 + 32,), -7, dtype=torch.int32, device="cuda")
    small = Buffers(w, 64)
    small.sendbuf = guard[:w.P * 64].view(w.P, 64)
    bls.bls_route_table_rr_static(small.rows, w.P, w.local_batch, torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda(),
                                  small.sendcounts, small.sdispls, small.sendbuf, small.sub_start, small.status)
    torch.cuda.synchronize()
    assert small.status.item() == 2
    assert torch.all(guard[w.P * 64:] == -7)
    assert int(small.sub_start.max()) <= 64
    off2 = off.copy()
    off2[5] = 2                                             # a bag that ends before it starts
    buf.route(w, ids, off2)
    assert buf.status.item() & 1
    buf.route(w, ids, off)                                  # and a good call afterwards is clean again
    check_against_oracle_and_plan(w, buf, ids, off)
    assert torch.ones(4, device="cuda").sum().item() == 4.0


def test_static_router_rejects_what_does_not_fit():
    lib = bls.lib()
    one = torch.zeros(4, dtype=torch.int32, device="cuda")
    rows = torch.ones(4000, dtype=torch.int64, device="cuda")
    p = lambda t: C.c_void_p(t.data_ptr())
    # P * (T + 1) = 32 * 4001 is beyond the static scratch: refused before any GPU work
    rc = lib.bls_route_table_rr_static(p(rows), 4000, 32, 1, p(one), p(one), C.c_int64(0), p(one), p(one), p(one),
                                       C.c_int64(4), p(one), p(one), None)
    assert rc == bls.BLS_ENOSPC
    rc = lib.bls_route_table_rr_static(p(rows), 4, 33, 1, p(one), p(one), C.c_int64(0), p(one), p(one), p(one),
                                       C.c_int64(4), p(one), p(one), None)
    assert rc == bls.BLS_EINVAL
