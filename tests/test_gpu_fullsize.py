"""Full-size workloads 2, 3, 4 and 5 in the configuration the benchmark times
(bls_step with the workload's largest bound, then the drain).

Routing artefacts of a whole iteration are compared with the oracle bit for
bit.  Pooled vectors: workloads 2 and 3 are compared in full, every one of the
53 248 / 425 984 vectors of the iteration; workloads 4 and 5 (33 GB and 64 GB
tables that never exist on the host) on 50 000 sampled bags plus every bag of
one whole (table, requester) chunk - which contains every boundary between the
runs the gather kernel cuts that chunk into - evaluated by the oracle one by
one from the counter-hash definition of the tables.  GPU only."""
import os

import numpy as np
import pytest
import torch

import bls_inputs as bi
import oracle
import paper_2512_19342_b200 as bls
from test_gpu_parity import TDT, TOL, check_route, dev_tables

pytestmark = pytest.mark.gpu
CORES = len(os.sched_getaffinity(0))


@pytest.mark.parametrize("num", [2, 3, 4, 5])
def test_full_size_iteration(num):
    w = bi.workload(num)
    need = w.table_bytes() * 1.25 + 8e9
    if torch.cuda.get_device_properties(0).total_memory < need:
        pytest.skip("not enough device memory for this workload")
    P, T, b, D = w.P, w.T, w.local_batch, w.tables[0].dim
    rng = np.random.Generator(np.random.PCG64(num))
    host_data = None
    if w.tables[0].kind == "hash":
        tabs = []
        for spec in w.tables:
            t = torch.empty(spec.rows, spec.dim, dtype=TDT[spec.dtype], device="cuda")
            bls.bls_fill_hash_table(t, spec.seed, spec.index)
            tabs.append(t)
        # the fill kernel against the generator, on rows spread over a table (first, last, random)
        spec = w.tables[T - 1]
        pick = np.unique(np.concatenate([[0, spec.rows - 1], rng.integers(0, spec.rows, 64)]))
        got = tabs[T - 1][torch.from_numpy(pick).cuda()].cpu()
        want = bi.hash_rows(spec.seed, spec.index, pick, spec.dim, spec.dtype)
        got = got.numpy() if spec.dtype == "f32" else got.view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(got, want.view(np.uint16) if spec.dtype == "f16" else want)
    else:
        host_data = [bi.table_values(t) for t in w.tables]
        tabs = dev_tables(w, host_data)

    ids, off = bi.make_iteration(w, 0)
    cap = int(np.diff(off[::T * b].astype(np.int64)).max()) + 64
    k = max(w.ks)
    plan = bls.bls_plan(tabs, w.partition, P, b, k, cap)
    bls.bls_set_poison(plan, True)                     # the slot starts as NaN: every bag must be written
    d_ids, d_off = torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda()
    out, it = bls.bls_step(plan, k, d_ids, d_off)
    assert (out is None) == (k > 0)
    view = bls.bls_view(plan, 0)
    # counts, displacements, packed buffers, sub-bag lengths; the receive-side counts exist once the
    # owners have answered (with a bound >= 1 that may be one step after the post, here: in the drain)
    check_route(w, view, ids, off, recv_side=min(bls.bls_counters(plan)[1]) > 0)
    while True:
        o, it = bls.bls_drain(plan)
        if o is None:
            break
        out = o
    check_route(w, view, ids, off)
    assert bls.bls_status(plan)[0] == bls.BLS_OK
    lens = np.diff(off.astype(np.int64))
    G = P * T * b
    if num in (2, 3):
        # the whole output, element by element (hash tables: rows evaluated on demand by the oracle)
        want = oracle.pool_definition(P, T, b, w.tables, host_data, ids, off, nthreads=CORES)
        got = out.cpu().numpy()
        err = oracle.vector_rel_err(got, want)
        assert err <= TOL[w.tables[0].dtype], err
    else:
        # 50 000 random bags, the longest, an empty one if any, the first and the last, and every
        # bag of one whole (requester, table) chunk, chosen at random
        src_c, t_c = int(rng.integers(P)), int(rng.integers(T))
        chunk = (src_c * T + t_c) * b + np.arange(b)
        sel = set(rng.integers(0, G, 50_000).tolist()) | {0, G - 1, int(lens.argmax()), int(lens.argmin())}
        sel = np.array(sorted(sel | set(chunk.tolist())), dtype=np.int64)
        want = oracle.pool_definition(P, T, b, w.tables, None, ids, off, sel=sel, nthreads=CORES)
        src, t, s = sel // (T * b), (sel // b) % T, sel % b
        got = out[torch.from_numpy(src).cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(t).cuda()].cpu().numpy()
        err = oracle.vector_rel_err(got, want)
        assert err <= TOL[w.tables[0].dtype], err
        empty = lens[sel] == 0
        assert np.all(got[empty] == 0)
    # properties that hold at any size: every bag written (no NaN left from the poison fill), totals consistent
    assert int(view["sendcounts"].sum()) == len(ids)
    assert torch.isfinite(out).all()
