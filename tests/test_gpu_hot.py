"""Hot-row staging: the selection follows the observed request counts, and the
staged path gives bit-identical pooled vectors and routing artefacts.  GPU only."""
import numpy as np
import pytest
import torch

import bls_inputs as bi
import oracle
import paper_2512_19342_b200 as bls
from test_gpu_parity import TOL, check_route, dev_tables, make_plan

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,mk,K", [
    ("cfg3_small", lambda: bi.workload(3, 0.02, 0.05), 96),
    ("cfg5_small", lambda: bi.workload(5, 0.001, 0.004), 40),
    ("uniform_few_rows", lambda: bi.tiny_workload(T=3, P=2, b=70, rows=50, dim=16, lengths="poisson10"), 64),
])
def test_staged_rows_change_nothing(name, mk, K):
    w = mk()
    data = [bi.table_values(t) for t in w.tables]
    tabs = dev_tables(w, data)
    P, T, b = w.P, w.T, w.local_batch
    plan_ref = make_plan(w, tabs, 1)
    plan_hot = make_plan(w, tabs, 1)
    bls.bls_hot_attach(plan_hot, K)
    observed = np.zeros((T, max(t.rows for t in w.tables)), np.int64)
    for it in (100, 101):                               # learn from batches that are not replayed below
        ids, off = bi.make_iteration(w, it)
        bls.bls_hot_observe(plan_hot, torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda())
        bag_table = (np.arange(P * T * b) // b) % T
        np.add.at(observed, (np.repeat(bag_table, np.diff(off)), ids), 1)
    bls.bls_hot_build(plan_hot)
    rows, count = bls.bls_hot_view(plan_hot)
    rows, count = rows.cpu().numpy(), count.cpu().numpy()
    for t in range(T):
        n = int(count[t])
        assert 0 <= n <= K
        sel = rows[t, :n]
        assert np.all(np.diff(sel) > 0)                 # slot order = row order, no duplicates
        cnt = observed[t]
        if n:
            thr = cnt[sel].min()
            assert thr >= 1
            rest = np.delete(cnt, sel)
            assert rest.max(initial=0) < thr            # every unselected row was requested less often
            # and the threshold could not be lowered by one without exceeding K slots
            assert n + np.count_nonzero(rest == rest.max(initial=0)) > K or rest.max(initial=0) == 0
    outs = {}
    for name_, plan in (("ref", plan_ref), ("hot", plan_hot)):
        got = []
        for it in range(3):
            ids, off = bi.make_iteration(w, it)
            out, oi = bls.bls_step(plan, 1, torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda())
            # the receive-side counts exist once the owners have answered the iteration
            check_route(w, bls.bls_view(plan, it), ids, off, recv_side=min(bls.bls_counters(plan)[1]) > it)
            if out is not None:
                got.append(out.clone())
        while True:
            out, oi = bls.bls_drain(plan)
            if out is None:
                break
            got.append(out.clone())
        assert bls.bls_status(plan)[0] == bls.BLS_OK and len(got) == 3
        outs[name_] = got
    for it in range(3):
        assert torch.equal(outs["ref"][it], outs["hot"][it])
        ids, off = bi.make_iteration(w, it)
        want = oracle.pool_definition(P, T, b, w.tables, data, ids, off)
        assert oracle.vector_rel_err(outs["hot"][it].cpu().numpy(), want) <= TOL[w.tables[0].dtype]


def test_hot_staging_is_refused_where_it_does_not_apply():
    w = bi.tiny_workload(T=2, P=2, b=4, rows=50, dim=8, partition="row_block")
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    plan = make_plan(w, tabs, 0, cap=64)
    with pytest.raises(bls.BlsError) as e:
        bls.bls_hot_attach(plan, 16)
    assert e.value.code == bls.BLS_ESTATE
    w = bi.tiny_workload(T=2, P=2, b=4, rows=50, dim=128)        # 512-byte rows: 1000 slots do not fit
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    plan = make_plan(w, tabs, 0, cap=64)
    with pytest.raises(bls.BlsError) as e:
        bls.bls_hot_attach(plan, 1000)
    assert e.value.code == bls.BLS_ENOSPC
