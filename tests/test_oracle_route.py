"""Pins for the oracle's routing artefacts (step 1), CPU only.

Each test fixes the oracle to something other than itself: a hand-enumerated
fixture, a closed form the paper states, or a library routine (numpy's stable
argsort and cumsum) that *is* the textbook alltoallv of bound k = 0
(Section III-D: with a zero bound the collective has the semantics of MPI_Alltoallv).
"""
import json
import os

import numpy as np
import pytest

import bls_inputs as bi
import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden", "route_tiny.json")


def _flat(bags):
    ids, off = [], [0]
    for rank in bags:
        for bag in rank:
            ids += bag
            off.append(len(ids))
    return np.array(ids, np.int32), np.array(off, np.int32)


@pytest.mark.parametrize("part", ["table_rr", "row_block"])
def test_hand_enumerated_fixture(part):
    g = json.load(open(GOLD))
    ids, off = _flat(g["bags"])
    art = oracle.route(g["P"], g["T"], g["b"], part, g["rows"], ids, off)
    for key, want in g[part].items():
        assert art[key].reshape(-1).tolist() == np.array(want).reshape(-1).tolist(), key


def _dst_local(w, ids, off):
    """Owner and owner-local row of every lookup (the two partitionings)."""
    P, T, b = w.P, w.T, w.local_batch
    lens = np.diff(off)
    bag = np.repeat(np.arange(len(lens)), lens)
    t = (bag // b) % T
    src = bag // (T * b)
    if w.partition == "table_rr":
        return src, t % P, ids.copy()
    rows = np.array([tb.rows for tb in w.tables])
    blk = -(-rows // P)
    d = ids // blk[t]
    return src, d, ids - d * blk[t]


@pytest.mark.parametrize("num,rs,bs", [(1, 1.0, 1.0), (2, 1.0, 1.0), (3, 0.01, 0.02),
                                       (4, 0.001, 0.004), (5, 0.001, 0.002)])
def test_against_numpy_stable_sort(num, rs, bs):
    w = bi.workload(num, rs, bs)
    ids, off = bi.make_iteration(w, 0)
    P, T, b = w.P, w.T, w.local_batch
    rows = [tb.rows for tb in w.tables]
    art = oracle.route(P, T, b, w.partition, rows, ids, off)
    src, dst, loc = _dst_local(w, ids, off)
    L = len(ids)
    # invariants the method fixes
    assert art["sendcounts"].sum() == L
    assert np.array_equal(art["recvcounts"], art["sendcounts"].T)
    excl = lambda m: np.cumsum(m, axis=1) - m
    assert np.array_equal(art["sdispls"], excl(art["sendcounts"]))
    assert np.array_equal(art["rdispls"], excl(art["recvcounts"]))
    # histogram by a library routine
    hist = np.zeros((P, P), np.int64)
    np.add.at(hist, (src, dst), 1)
    assert np.array_equal(hist, art["sendcounts"])
    # packed send buffer = stable sort by (src, dst): numpy's stable argsort
    order = np.argsort(src * P + dst, kind="stable")
    assert np.array_equal(art["sendbuf"], loc[order])
    # receive buffer = the same lookups stably sorted by (dst, src)
    order_r = np.argsort(dst * P + src, kind="stable")
    assert np.array_equal(art["recvbuf"], loc[order_r])
    # the route is a permutation of the requests
    assert np.array_equal(np.sort(art["sendbuf"]), np.sort(loc))
    # sub-bag lengths add up to the receive counts, pair by pair
    pos = 0
    for d in range(P):
        per = oracle.subbags_per_pair(w.partition, P, T, b, d)
        for s in range(P):
            assert art["sublen"][pos:pos + per].sum() == art["recvcounts"][d, s]
            pos += per
    assert pos == len(art["sublen"])


def test_onehot_tablewise_closed_form():
    """One ID per table per sample and table-wise placement give message sizes
    that differ only through the table count per rank (Section V-E, setting 1,
    last sentence): sendcounts[src][dst] = b * ntables(dst)."""
    w1 = bi.workload(1)
    ids, off = bi.make_iteration(w1, 3)
    a = oracle.route(w1.P, w1.T, w1.local_batch, "table_rr", [t.rows for t in w1.tables], ids, off)
    assert np.all(a["sendcounts"] == 128)
    w2 = bi.workload(2)
    ids, off = bi.make_iteration(w2, 5)
    a = oracle.route(w2.P, w2.T, w2.local_batch, "table_rr", [t.rows for t in w2.tables], ids, off)
    want = np.where(np.arange(8) < 2, 1024, 768)
    assert np.array_equal(a["sendcounts"], np.tile(want, (8, 1)))


def test_uniform_rowwise_counts_are_balanced():
    w = bi.tiny_workload(T=4, P=4, b=64, rows=4000, partition="row_block", lengths="poisson10")
    ids, off = bi.make_iteration(w, 0)
    a = oracle.route(4, 4, 64, "row_block", [4000] * 4, ids, off)
    L = len(ids)
    mean = L / 16
    assert np.all(np.abs(a["sendcounts"] - mean) < 6 * np.sqrt(mean))   # binomial bound


def test_empty_and_degenerate_inputs():
    # all bags empty
    off = np.zeros(2 * 3 * 2 + 1, np.int32)
    a = oracle.route(2, 3, 2, "table_rr", [4, 6, 5], np.zeros(0, np.int32), off)
    assert a["sendcounts"].sum() == 0 and np.all(a["sublen"] == 0)
    # single rank: everything is local, send buffer is the id list itself
    w = bi.tiny_workload(T=3, P=1, b=5, rows=9)
    ids, off = bi.make_iteration(w, 1)
    a = oracle.route(1, 3, 5, "row_block", [9] * 3, ids, off)
    assert np.array_equal(a["sendbuf"], ids) and np.array_equal(a["recvbuf"], ids)
    assert np.array_equal(a["sublen"], np.diff(off))


def test_out_of_range_id_is_reported():
    ids, off = np.array([0, 7], np.int32), np.array([0, 1, 2], np.int32)
    with pytest.raises(ValueError):
        oracle.route(1, 1, 2, "table_rr", [7], ids, off)
