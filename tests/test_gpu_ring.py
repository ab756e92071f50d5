"""The BLS slot ring on the GPU: output for any bound k equals the synchronous
output (Abstract: the bound does not change what is computed; Section III-D: k = 0 is the plain
alltoallv), ranks really lag under injected delays, never by more than k, and a
wait that cannot end in time returns a status instead of hanging.  GPU only."""
import numpy as np
import pytest
import torch

import bls_inputs as bi
import oracle
import paper_2512_19342_b200 as bls
from test_gpu_parity import TOL, check_route, dev_tables, make_plan

pytestmark = pytest.mark.gpu


def assert_matches_oracle(w, data, inputs, outs):
    """Every handed-back iteration against the oracle's pooled output by definition."""
    for it, (ids, off) in enumerate(inputs):
        want = oracle.pool_definition(w.P, w.T, w.local_batch, w.tables, data, ids, off)
        err = oracle.vector_rel_err(outs[it].cpu().numpy(), want)
        assert err <= TOL[w.tables[0].dtype], (it, err)


def run_loop(w, tabs, k, n_iter, k_max=None, stalls=None, check_views=False, wait_limit=None):
    """Listing 2's loop: n_iter steps then the drain; returns {iteration: output}."""
    plan = make_plan(w, tabs, k if k_max is None else k_max)
    if wait_limit is not None:
        bls.bls_set_wait_limit(plan, wait_limit)
    for r, ns in (stalls or {}).items():
        bls.bls_set_stall(plan, r, ns)
    outs, inputs = {}, []
    for t in range(n_iter):
        ids, off = bi.make_iteration(w, t)
        inputs.append((ids, off))
        d_ids, d_off = torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda()
        out, it = bls.bls_step(plan, k, d_ids, d_off)
        if t < k:
            assert out is None and it == -1
        else:
            assert it == t - k
            outs[it] = out.clone()
        if check_views and not stalls:
            # with a bound >= 1 the owners may answer an iteration one step after it was posted
            served = bls.bls_counters(plan)[1]
            check_route(w, bls.bls_view(plan, t), ids, off, recv_side=min(served) > t)
    while True:
        out, it = bls.bls_drain(plan)
        if out is None:
            break
        assert it == len(outs)                    # oldest first
        outs[it] = out.clone()
    if check_views and not stalls:
        check_route(w, bls.bls_view(plan, n_iter - 1), *inputs[-1])
    status, lag = bls.bls_status(plan)
    posted, served, done = bls.bls_counters(plan)
    assert posted == served == done == [n_iter] * w.P
    return outs, inputs, status, lag


@pytest.mark.parametrize("num,rs,bs", [(1, 1.0, 1.0), (3, 0.01, 0.02), (4, 0.002, 0.01)])
def test_output_is_independent_of_k(num, rs, bs):
    w = bi.workload(num, rs, bs)
    data = [bi.table_values(t) for t in w.tables]
    tabs = dev_tables(w, data)
    n_iter = 7
    ref, inputs, status, lag = run_loop(w, tabs, 0, n_iter, check_views=True)
    assert status == bls.BLS_OK and lag == 0 and sorted(ref) == list(range(n_iter))
    P, T, b = w.P, w.T, w.local_batch
    for it, (ids, off) in enumerate(inputs):
        want = oracle.pool_definition(P, T, b, w.tables, data, ids, off)
        assert oracle.vector_rel_err(ref[it].cpu().numpy(), want) <= TOL[w.tables[0].dtype]
    for k in (1, 2, 4, 8):
        outs, _, status, lag = run_loop(w, tabs, k, n_iter, check_views=True)
        assert status == bls.BLS_OK and lag <= k
        assert sorted(outs) == list(range(n_iter))
        for it in range(n_iter):
            assert torch.equal(outs[it], ref[it]), (k, it)           # deterministic kernels: bit-identical


def test_ring_larger_than_bound():
    """A plan made for k_max = 4 also serves k = 1 (fewer slots in flight)."""
    w = bi.workload(1)
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    ref, *_ = run_loop(w, tabs, 0, 5)
    outs, _, status, _ = run_loop(w, tabs, 1, 5, k_max=4)
    assert status == bls.BLS_OK
    assert all(torch.equal(outs[i], ref[i]) for i in range(5))


@pytest.mark.parametrize("part", ["table_rr", "row_block"])
def test_delayed_ranks_lag_within_the_bound(part):
    """Injected delays (Section V-E, setting 2) make ranks fall behind; the
    counters keep them within k iterations and the results do not change."""
    w = bi.tiny_workload(T=4, P=4, b=64, rows=500, dim=16, partition=part, lengths="poisson10")
    data = [bi.table_values(t) for t in w.tables]
    tabs = dev_tables(w, data)
    n_iter = 10
    ref, inputs, *_ = run_loop(w, tabs, 0, n_iter)
    assert_matches_oracle(w, data, inputs, ref)
    for k in (1, 3):
        outs, _, status, lag = run_loop(w, tabs, k, n_iter, stalls={1: 3_000_000, 2: 500_000})
        assert status == bls.BLS_OK
        assert 1 <= lag <= k, lag                                     # somebody really ran ahead
        assert_matches_oracle(w, data, inputs, outs)
        for it in range(n_iter):
            assert torch.equal(outs[it], ref[it]), (k, it)
    # bound 0: the delay is paid every iteration, nobody runs ahead
    outs, _, status, lag = run_loop(w, tabs, 0, 4, stalls={1: 1_000_000})
    assert status == bls.BLS_OK and lag == 0
    assert_matches_oracle(w, data, inputs[:4], outs)
    assert all(torch.equal(outs[i], ref[i]) for i in range(4))


def test_wait_that_cannot_end_returns_a_status():
    """A delay longer than the wait limit: the gate gives up, records
    BLS_ETIMEOUT, goes on with correct data, and the context stays usable."""
    w = bi.workload(1)
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    ref, *_ = run_loop(w, tabs, 0, 3)
    outs, _, status, _ = run_loop(w, tabs, 0, 3, stalls={0: 5_000_000_000}, wait_limit=200_000)
    assert status == bls.BLS_ETIMEOUT
    assert all(torch.equal(outs[i], ref[i]) for i in range(3))
    assert torch.ones(8, device="cuda").sum().item() == 8.0


def test_bound_of_one_or_more_routes_beside_the_previous_answer():
    """Table-wise placement, bound >= 1, no delays: a step posts iteration t and answers
    iteration t - 1 (the router runs beside the gather kernel), so after a step the owners
    are one iteration behind the requesters and the drain catches up."""
    w = bi.workload(2, 0.05, 0.25)
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    plan = make_plan(w, tabs, 2)
    for t in range(3):
        ids, off = bi.make_iteration(w, t)
        bls.bls_step(plan, 2, torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda())
        posted, served, done = bls.bls_counters(plan)
        assert posted == [t + 1] * w.P and served == [t] * w.P and done == [t] * w.P
    out, it = bls.bls_drain(plan)
    assert it == 1
    posted, served, done = bls.bls_counters(plan)
    assert posted == served == done == [3] * w.P
    assert bls.bls_status(plan) == (bls.BLS_OK, 1)


def test_delays_switched_on_and_off_mid_flight():
    """A loop that starts in overlapped mode (bound 2, no delays), gets a delayed rank after
    three steps (from then on the plan works in waves on one stream) and loses the delay again
    after six: the owners' one-iteration backlog is carried over, every iteration comes back
    once, in order, unchanged."""
    w = bi.workload(2, 0.05, 0.25)
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    n_iter = 9
    ref, inputs, *_ = run_loop(w, tabs, 0, n_iter)
    plan = make_plan(w, tabs, 2)
    got = []
    for t, (ids, off) in enumerate(inputs):
        if t == 3:
            bls.bls_set_stall(plan, 1, 400_000)
        if t == 6:
            bls.bls_set_stall(plan, 1, 0)
        out, it = bls.bls_step(plan, 2, torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda())
        if out is not None:
            assert it == len(got)
            got.append(out.clone())
    while True:
        out, it = bls.bls_drain(plan)
        if out is None:
            break
        assert it == len(got)
        got.append(out.clone())
    status, lag = bls.bls_status(plan)
    assert status == bls.BLS_OK and lag <= 2 and len(got) == n_iter
    assert all(torch.equal(got[i], ref[i]) for i in range(n_iter))
    posted, served, done = bls.bls_counters(plan)
    assert posted == served == done == [n_iter] * w.P


def test_changing_k_mid_flight_is_refused():
    w = bi.workload(1)
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    plan = make_plan(w, tabs, 2)
    ids, off = bi.make_iteration(w, 0)
    d_ids, d_off = torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda()
    bls.bls_step(plan, 2, d_ids, d_off)
    with pytest.raises(bls.BlsError) as e:
        bls.bls_step(plan, 1, d_ids, d_off)
    assert e.value.code == bls.BLS_ESTATE
    while bls.bls_drain(plan)[0] is not None:
        pass
    out, it = bls.bls_step(plan, 0, d_ids, d_off)              # allowed again after the drain
    assert it == 1 and out is not None


def test_host_buffer_entry_points():
    """bls_step_host / bls_drain_host: host IDs in, host vectors out."""
    w = bi.workload(3, 0.01, 0.02)
    data = [bi.table_values(t) for t in w.tables]
    tabs = dev_tables(w, data)
    plan = make_plan(w, tabs, 1)
    P, T, b, D = w.P, w.T, w.local_batch, w.tables[0].dim
    host_out = torch.empty(P, b, T, D, dtype=torch.float32).pin_memory()
    got, inputs = {}, []
    for t in range(4):
        ids, off = bi.make_iteration(w, t)
        inputs.append((ids, off))
        it = bls.bls_step_host(plan, 1, torch.from_numpy(ids).pin_memory(), torch.from_numpy(off).pin_memory(), host_out)
        torch.cuda.synchronize()
        if it >= 0:
            got[it] = host_out.clone()
    while True:
        it = bls.bls_drain_host(plan, host_out)
        torch.cuda.synchronize()
        if it < 0:
            break
        got[it] = host_out.clone()
    assert sorted(got) == [0, 1, 2, 3] and bls.bls_status(plan)[0] == bls.BLS_OK
    for it, (ids, off) in enumerate(inputs):
        want = oracle.pool_definition(P, T, b, w.tables, data, ids, off)
        assert oracle.vector_rel_err(got[it].numpy(), want) <= 1e-5


def test_random_delays_are_masked_by_the_bound():
    """Section V-E setting 2 / Section VI-B: every rank is delayed by a uniform random time
    before each iteration.  Bound 0 pays the largest of the P delays in every iteration;
    a bound k > 0 lets ranks drift apart and hides part of it.  Results do not change."""
    w = bi.tiny_workload(T=4, P=4, b=64, rows=500, dim=16, lengths="poisson10")
    data = [bi.table_values(t) for t in w.tables]
    tabs = dev_tables(w, data)
    n_iter, span = 40, 400_000                                  # delays uniform in [0, 400 us]
    inputs = [bi.make_iteration(w, t) for t in range(n_iter)]
    d_in = [(torch.from_numpy(i).cuda(), torch.from_numpy(o).cuda()) for i, o in inputs]
    times, outs = {}, {}
    for k in (0, 4):
        plan = make_plan(w, tabs, k)
        for r in range(w.P):
            bls.bls_set_random_stall(plan, r, span, seed=1234)
        bls.bls_set_waves_per_step(plan, w.P + 1)               # one wave per rank that may act, plus the forcing one
        got = []
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for t in range(n_iter):
            out, it = bls.bls_step(plan, k, *d_in[t])
            if out is not None:
                got.append(out.clone())
        while True:
            out, it = bls.bls_drain(plan)
            if out is None:
                break
            got.append(out.clone())
        e1.record()
        torch.cuda.synchronize()
        status, lag = bls.bls_status(plan)
        assert status == bls.BLS_OK and lag <= k and len(got) == n_iter
        assert_matches_oracle(w, data, inputs, got)
        times[k], outs[k] = e0.elapsed_time(e1) / n_iter, got
    assert all(torch.equal(a, b) for a, b in zip(outs[0], outs[4]))
    # bound 0: about the mean of the maximum of four delays (320 us) per iteration
    assert times[0] > 0.25
    assert times[4] < 0.9 * times[0], times


def test_largest_ring():
    """k_max = 15 (16 slots) and 32 ranks, the limits of a plan."""
    w = bi.tiny_workload(T=6, P=32, b=3, rows=50, dim=8, lengths="mixed")
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    ref, *_ = run_loop(w, tabs, 0, 20)
    outs, _, status, lag = run_loop(w, tabs, 15, 20, check_views=True)
    assert status == bls.BLS_OK and lag <= 1       # no delays: at most the one iteration that is routed beside the answer of the previous one
    assert all(torch.equal(outs[i], ref[i]) for i in range(20))
    outs, _, status, lag = run_loop(w, tabs, 15, 20, stalls={5: 6_000_000, 31: 1_000_000})   # longer than a host step
    assert status == bls.BLS_OK and 1 <= lag <= 15
    assert all(torch.equal(outs[i], ref[i]) for i in range(20))
