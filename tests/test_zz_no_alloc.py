"""bls_route_table_rr_static: the router for callers that cannot allocate device
memory (a process whose GPU memory belongs to another framework's pool, a plugin
with fixed buffers).  Its scratch is a static device array shared by all calls,
so the test calls it twice in a row with different inputs and compares every
output, bit for bit, with the plan-based router (bls_route + bls_view).  This
file is collected last on purpose.  GPU only."""
import numpy as np
import pytest
import torch

import bls_inputs as bi
import paper_2512_19342_b200 as bls

pytestmark = pytest.mark.gpu


def test_static_router_matches_plan_router_twice_in_a_row():
    w = bi.workload(3, 0.02, 0.03)                      # 26 tables, P=8, b=61, bags of about 20 IDs
    P, T, b = w.P, w.T, w.local_batch
    tabs = [torch.empty(t.rows, t.dim, device="cuda") for t in w.tables]   # values are not read by the router
    inputs = [bi.make_iteration(w, it) for it in (0, 1)]
    cap = max(int(np.diff(off[::T * b].astype(np.int64)).max()) for _, off in inputs) + 13
    cap = (cap + 3) // 4 * 4
    plan = bls.bls_plan(tabs, "table_rr", P, b, 0, cap)
    # the caller's buffers for the static entry point, allocated once up front
    rows = torch.tensor([t.rows for t in w.tables], dtype=torch.int64, device="cuda")
    sendcounts = torch.empty(P, P, dtype=torch.int32, device="cuda")
    sdispls = torch.empty(P, P, dtype=torch.int32, device="cuda")
    sendbuf = torch.empty(P, cap, dtype=torch.int32, device="cuda")
    sub_start = torch.empty(P, T * b + 1, dtype=torch.int32, device="cuda")
    status = torch.empty(1, dtype=torch.int32, device="cuda")
    for it, (ids, off) in enumerate(inputs):
        d_ids, d_off = torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda()
        sendbuf.fill_(-7)
        bls.bls_route_table_rr_static(rows, P, b, d_ids, d_off, sendcounts, sdispls, sendbuf, sub_start, status)
        bls.bls_route(plan, it, d_ids, d_off)
        ref = bls.bls_view(plan, it)
        torch.cuda.synchronize()
        assert status.item() == 0
        assert torch.equal(sendcounts, ref["sendcounts"])
        assert torch.equal(sdispls, ref["sdispls"])
        assert torch.equal(sub_start, ref["sub_start"])
        per_rank = np.diff(off[::T * b].astype(np.int64))
        for src in range(P):
            n = int(per_rank[src])
            assert torch.equal(sendbuf[src, :n], ref["sendbuf"][src, :n]), (it, src)
            assert torch.all(sendbuf[src, n:] == -7)             # nothing written past the rank's total
        bls.bls_lookup(plan, it)
    assert bls.bls_status(plan)[0] == bls.BLS_OK


def test_static_router_rejects_what_does_not_fit():
    lib = bls.lib()
    import ctypes as C
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
