"""Small table-wise iterations in one kernel launch (bls_set_fused): routing artefacts bit for bit
and pooled vectors within tolerance against the oracle, bit-identical to the stand-alone kernels,
the ring's counters and time stamps advance as in a wave, bad inputs are reported, and the mode
hands over to the other modes in the middle of a plan's life.  GPU only."""
import numpy as np
import pytest
import torch

import bls_inputs as bi
import oracle
import paper_2512_19342_b200 as bls
from test_gpu_parity import CASES, TOL, check_route, dev_tables, make_plan

pytestmark = pytest.mark.gpu

TABLE_WISE = [name for name, mk in CASES if mk().partition == "table_rr"]


def fused_plan(w, tabs, k_max, cap=None):
    plan = make_plan(w, tabs, k_max, cap)
    bls.bls_set_overlap(plan, -1)
    bls.bls_set_fused(plan, 1)
    return plan


@pytest.mark.parametrize("k", [0, 2])
@pytest.mark.parametrize("name", TABLE_WISE)
def test_one_launch_iterations_match_oracle_and_kernels(name, k):
    w = dict(CASES)[name]()
    data = [bi.table_values(t) for t in w.tables]
    tabs = dev_tables(w, data)
    plan, ref_plan = fused_plan(w, tabs, k), make_plan(w, tabs, 0)
    bls.bls_profile(plan, True)
    n_iter, inputs, outs = 5, [], {}
    for t in range(n_iter):
        ids, off = bi.make_iteration(w, t)
        inputs.append((ids, off))
        d_ids, d_off = torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda()
        out, it = bls.bls_step(plan, k, d_ids, d_off)
        assert it == (t - k if t >= k else -1)
        if out is not None:
            outs[it] = out.clone()
        # the iteration is complete on every rank when the launch ends
        assert bls.bls_counters(plan) == ([t + 1] * w.P,) * 3
        view = bls.bls_view(plan, t)
        check_route(w, view, ids, off)
        # the stand-alone kernels on the same inputs: same bits
        ref_out, _ = bls.bls_step(ref_plan, 0, d_ids, d_off)
        assert torch.equal(view["out"], ref_out), (name, t)
        ref_view = bls.bls_view(ref_plan, t)
        for key in ("sendcounts", "sdispls", "recvcounts", "rdispls", "sendbuf", "sub_start"):
            got, want = view[key], ref_view[key]
            if key == "sendbuf":                       # beyond a rank's count the buffer holds leftovers
                for src in range(w.P):
                    n = int(view["sendcounts"][src].sum())
                    assert torch.equal(got[src, :n], want[src, :n])
            else:
                assert torch.equal(got, want), key
    while True:
        out, it = bls.bls_drain(plan)
        if out is None:
            break
        assert it == len(outs)
        outs[it] = out.clone()
    assert sorted(outs) == list(range(n_iter))
    for it, (ids, off) in enumerate(inputs):
        want = oracle.pool_definition(w.P, w.T, w.local_batch, w.tables, data, ids, off)
        assert oracle.vector_rel_err(outs[it].cpu().numpy(), want) <= TOL[w.tables[0].dtype], (name, it)
    status, lag = bls.bls_status(plan)
    assert status == bls.BLS_OK and lag == 0
    assert bls.bls_profile_read(plan)["kernels_total"] == n_iter        # one launch per iteration, none for the drain


def test_default_plan_uses_one_launch_for_small_iterations_only():
    """Mode 0 (the default): the paper's small one-ID-per-table shapes take the one-launch kernel,
    a plan with room for 256 K lookups or more per iteration takes the wave of kernels."""
    w = bi.workload(1)
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    for cap, per_step in ((w.T * w.local_batch, 1), (1 << 16, 3)):
        plan = bls.bls_plan(tabs, w.partition, w.P, w.local_batch, 0, cap)
        before = bls.bls_profile_read(plan)["kernels_total"]
        for t in range(4):
            ids, off = bi.make_iteration(w, t)
            bls.bls_step(plan, 0, torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda())
        assert bls.bls_profile_read(plan)["kernels_total"] - before == 4 * per_step
        assert bls.bls_status(plan)[0] == bls.BLS_OK


def test_time_stamps_of_one_launch_iterations():
    w = bi.workload(2, 0.05, 0.25)
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    plan = fused_plan(w, tabs, 1)
    n = 6
    for t in range(n):
        ids, off = bi.make_iteration(w, t)
        bls.bls_step(plan, 1, torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda())
    while bls.bls_drain(plan)[0] is not None:
        pass
    post, serve, done = bls.bls_timeline(plan, 0, n)
    assert (post > 0).all() and np.array_equal(post, serve) and np.array_equal(post, done)
    assert (np.diff(post.astype(np.int64), axis=0) > 0).all()           # one iteration after the other
    assert (post == post[:, :1]).all()                                 # all ranks of a launch together


def test_hands_over_to_the_other_modes():
    """One plan: one-launch iterations, then route + lookup, then injected delays (the persistent ring
    kernel), then stand-alone waves; every iteration against the oracle."""
    w = bi.tiny_workload(T=5, P=3, b=70, rows=400, dim=16, lengths="poisson10")
    data = [bi.table_values(t) for t in w.tables]
    tabs = dev_tables(w, data)
    plan = fused_plan(w, tabs, 2)
    t = 0

    def check(out, it):
        ids, off = bi.make_iteration(w, it)
        want = oracle.pool_definition(w.P, w.T, w.local_batch, w.tables, data, ids, off)
        assert oracle.vector_rel_err(out.cpu().numpy(), want) <= 1e-5, it

    def loop(k, n):
        nonlocal t
        handed = []
        for _ in range(n):
            ids, off = bi.make_iteration(w, t)
            out, it = bls.bls_step(plan, k, torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda())
            t += 1
            if out is not None:
                check(out, it)
                handed.append(it)
        while True:
            out, it = bls.bls_drain(plan)
            if out is None:
                break
            check(out, it)
            handed.append(it)
        assert handed == list(range(t - n, t))

    loop(2, 4)                                             # one launch per iteration
    ids, off = bi.make_iteration(w, t)
    bls.bls_route(plan, t, torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda())
    bls.bls_lookup(plan, t)
    check(bls.bls_view(plan, t)["out"], t)
    t += 1
    loop(0, 2)                                             # one launch again
    loop(1, 3)
    bls.bls_set_fused(plan, -1)
    loop(0, 2)                                             # waves of stand-alone kernels
    bls.bls_set_overlap(plan, 1)
    loop(2, 3)                                             # ... the router beside the previous answer
    bls.bls_set_overlap(plan, -1)
    bls.bls_set_fused(plan, 1)
    loop(2, 3)
    assert bls.bls_status(plan) == (bls.BLS_OK, 1)         # (the overlapped waves are one iteration apart)
    bls.bls_set_stall(plan, 1, 1_000_000)
    loop(2, 4)                                             # persistent ring kernel, rank 1 behind
    status, lag = bls.bls_status(plan)
    assert status == bls.BLS_OK and lag == 2
    assert bls.bls_counters(plan) == ([t] * w.P,) * 3


def test_bad_inputs_are_reported_by_the_one_launch_kernel():
    w = bi.tiny_workload(T=2, P=2, b=3, rows=10, dim=8, lengths="one")
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    ids, off = bi.make_iteration(w, 0)
    bad = ids.copy()
    bad[3] = 10
    bad[5] = -1
    plan = fused_plan(w, tabs, 0, cap=64)
    out, _ = bls.bls_step(plan, 0, torch.from_numpy(bad).cuda(), torch.from_numpy(off).cuda())
    assert bls.bls_status(plan)[0] == bls.BLS_ERANGE
    assert torch.isfinite(out).all()
    # a send buffer that is too small
    plan = fused_plan(w, tabs, 0, cap=2)
    bls.bls_step(plan, 0, torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda())
    assert bls.bls_status(plan)[0] == bls.BLS_ENOSPC
    # offsets that go backwards
    boff = off.copy()
    boff[4] = 1
    plan = fused_plan(w, tabs, 0, cap=64)
    bls.bls_step(plan, 0, torch.from_numpy(ids).cuda(), torch.from_numpy(boff).cuda())
    assert bls.bls_status(plan)[0] == bls.BLS_EINVAL
    assert torch.ones(8, device="cuda").sum().item() == 8.0


def test_all_bags_empty_in_one_launch():
    w = bi.tiny_workload(T=3, P=2, b=4, rows=9, dim=16)
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    plan = fused_plan(w, tabs, 0, cap=8)
    off = torch.zeros(2 * 3 * 4 + 1, dtype=torch.int32, device="cuda")
    ids = torch.zeros(0, dtype=torch.int32, device="cuda")
    out, it = bls.bls_step(plan, 0, ids, off)
    assert it == 0 and bls.bls_status(plan)[0] == bls.BLS_OK
    assert torch.count_nonzero(out).item() == 0
    assert int(bls.bls_view(plan, 0)["sendcounts"].sum()) == 0
