"""CUDA path vs CPU oracle, element by element, through the C ABI.  GPU only.

Bars: routing artefacts (counts, displacements, packed buffers, sub-bag
lengths) bit-exact; pooled vectors within max relative error 1e-5 (fp32
tables) / 1e-2 (bf16, fp16 tables), measured per output vector as
max_c|g-o| / max_c|o|.
"""
import numpy as np
import pytest
import torch

import bls_inputs as bi
import oracle
import paper_2512_19342_b200 as bls

pytestmark = pytest.mark.gpu
TOL = {"f32": 1e-5, "bf16": 1e-2, "f16": 1e-2}
TDT = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}


def dev_tables(w, data):
    out = []
    for spec, d in zip(w.tables, data):
        t = torch.from_numpy(d.view(np.int16) if spec.dtype == "bf16" else d)
        t = t.view(torch.bfloat16) if spec.dtype == "bf16" else t
        out.append(t.cuda().contiguous())
    return out


def make_plan(w, tabs, k_max, cap=None):
    if cap is None:
        cap = 1
        for it in range(6):
            ids, off = bi.make_iteration(w, it)
            per = np.diff(off[::w.T * w.local_batch].astype(np.int64))
            cap = max(cap, int(per.max()))
        cap = int(cap * 1.25) + 16
    plan = bls.bls_plan(tabs, w.partition, w.P, w.local_batch, k_max, cap)
    bls.bls_set_poison(plan, True)          # every bag must be written: an unwritten one would show up as NaN
    bls.bls_set_overlap(plan, 1)            # test workloads are small: use the overlapped mode wherever it applies
    bls.bls_set_fused(plan, -1)             # ... and the stand-alone kernels, not the one-launch kernel for small iterations,
    return plan                             # which has tests of its own (test_gpu_fused.py)


def check_route(w, view, ids, off, recv_side=True):
    """Device routing artefacts of one iteration against the oracle, bit for bit.
    The receive-side counts exist once the owners have answered the iteration."""
    P, T, b = w.P, w.T, w.local_batch
    art = oracle.route(P, T, b, w.partition, [t.rows for t in w.tables], ids, off)
    for key in ("sendcounts", "sdispls") + (("recvcounts", "rdispls") if recv_side else ()):
        assert np.array_equal(view[key].cpu().numpy(), art[key]), key
    sendbuf = view["sendbuf"].cpu().numpy()
    sub = view["sub_start"].cpu().numpy()
    base = off[::T * b]
    recv_parts = {}
    for src in range(P):
        n = int(base[src + 1] - base[src])
        assert np.array_equal(sendbuf[src, :n], art["sendbuf"][base[src]:base[src + 1]]), f"sendbuf of rank {src}"
        if not view["sub_bag_major"]:
            assert sub[src, -1] == n and sub[src, 0] == 0
        for d in range(P):
            lo = art["sdispls"][src, d]
            recv_parts[(d, src)] = sendbuf[src, lo:lo + art["sendcounts"][src, d]]
    # what owner d receives (segments at rdispls) equals the oracle's receive buffer
    recv = np.concatenate([recv_parts[(d, s)] for d in range(P) for s in range(P)]) if len(ids) else np.zeros(0, np.int32)
    assert np.array_equal(recv, art["recvbuf"])
    # sub-bag lengths in (dst, src, bag) order
    got, pos = [], 0
    if view["sub_bag_major"]:                      # row-wise: entries ordered (table, sample, dst)
        s3 = sub.astype(np.int64).reshape(P, T * b + 1, P)
        assert np.array_equal(s3[:, 0, :], art["sdispls"])
        assert np.array_equal(s3[:, -1, :], art["sdispls"] + art["sendcounts"])
        lens3 = np.diff(s3, axis=1)                # [src][bag][dst]
        for d in range(P):
            for src in range(P):
                got.append(lens3[src, :, d])
    else:
        lens = np.diff(sub.astype(np.int64), axis=1)
        for d in range(P):
            per = oracle.subbags_per_pair(w.partition, P, T, b, d)
            for src in range(P):
                got.append(lens[src, pos:pos + per])
            pos += per
    assert np.array_equal(np.concatenate(got), art["sublen"])
    return art


CASES = [
    ("cfg1", lambda: bi.workload(1)),
    ("cfg2_small", lambda: bi.workload(2, 0.05, 0.25)),
    ("cfg3_small", lambda: bi.workload(3, 0.02, 0.03)),          # b=61: ragged tiles, 20-id bags
    ("cfg4_small", lambda: bi.workload(4, 0.002, 0.01)),         # row-wise bf16, b=20
    ("cfg5_small", lambda: bi.workload(5, 0.001, 0.003)),        # fp16, P=32, b=6
    ("tiny_rr", lambda: bi.tiny_workload(T=3, P=2, b=2, rows=[4, 6, 5], dim=4)),
    ("tiny_rb", lambda: bi.tiny_workload(T=3, P=2, b=2, rows=[4, 6, 5], dim=4, partition="row_block")),
    ("more_ranks_than_tables", lambda: bi.tiny_workload(T=2, P=5, b=3, rows=50, dim=8)),
    ("rows_fewer_than_ranks", lambda: bi.tiny_workload(T=2, P=4, b=130, rows=3, dim=8, partition="row_block")),
    ("one_rank", lambda: bi.tiny_workload(T=4, P=1, b=300, rows=1000, dim=32, lengths="poisson20c")),
    ("wide_rows_bf16", lambda: bi.tiny_workload(T=3, P=3, b=129, rows=500, dim=256, dtype="bf16",
                                                partition="row_block", lengths="poisson10")),
    ("narrow_rows", lambda: bi.tiny_workload(T=3, P=2, b=257, rows=100, dim=4, lengths="pareto15c")),
    ("dim128_f32", lambda: bi.tiny_workload(T=2, P=2, b=40, rows=300, dim=128, lengths="poisson20c")),
    ("f16_dim8", lambda: bi.tiny_workload(T=5, P=3, b=33, rows=77, dim=8, dtype="f16", lengths="mixed")),
    ("extreme_bags", lambda: bi.tiny_workload(T=3, P=2, b=50, rows=300, dim=64, lengths="extremes")),
    ("extreme_bags_rowwise", lambda: bi.tiny_workload(T=3, P=4, b=50, rows=300, dim=32, dtype="f16",
                                                      partition="row_block", lengths="extremes")),
    ("long_bags_rowwise", lambda: bi.tiny_workload(T=2, P=3, b=130, rows=900, dim=16, partition="row_block",
                                                   lengths="extremes")),    # two tiles per table, thousands of lookups per tile
    ("rowwise_wide_tiles", lambda: bi.tiny_workload(T=8, P=8, b=4096, rows=5000, dim=8, partition="row_block",
                                                    lengths="poisson10")),   # tiles of 256 bags, routed in two passes each
    ("short_bags_wide_tiles", lambda: bi.tiny_workload(T=9, P=4, b=700, rows=50, dim=8, lengths="pareto15c")),  # table-wise tiles of 256+ bags
    ("many_tables", lambda: bi.tiny_workload(T=70, P=3, b=9, rows=40, dim=16, lengths="mixed")),           # > 32 (owner, table) pairs
    ("max_ranks", lambda: bi.tiny_workload(T=40, P=32, b=5, rows=64, dim=32, lengths="poisson10")),
    ("max_ranks_rowwise", lambda: bi.tiny_workload(T=3, P=32, b=7, rows=1000, dim=64, dtype="bf16",
                                                   partition="row_block", lengths="poisson20c")),
    ("rowwise_more_ranks_than_lanes", lambda: bi.tiny_workload(T=4, P=12, b=20, rows=300, dim=16,
                                                               partition="row_block", lengths="poisson10")),  # 4 lanes, 12 owners
]


@pytest.mark.parametrize("name,mk", CASES, ids=[c[0] for c in CASES])
def test_route_and_lookup_match_oracle(name, mk):
    w = mk()
    data = [bi.table_values(t) for t in w.tables]
    tabs = dev_tables(w, data)
    plan = make_plan(w, tabs, k_max=0)
    P, T, b = w.P, w.T, w.local_batch
    for it in range(3):
        ids, off = bi.make_iteration(w, it)
        d_ids, d_off = torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda()
        bls.bls_route(plan, it, d_ids, d_off)
        view = bls.bls_view(plan, it)
        bls.bls_lookup(plan, it)
        st, _ = bls.bls_status(plan)
        assert st == bls.BLS_OK
        check_route(w, view, ids, off)
        want = oracle.pool_definition(P, T, b, w.tables, data, ids, off)
        got = view["out"].cpu().numpy()
        err = oracle.vector_rel_err(got, want)
        assert err <= TOL[w.tables[0].dtype], (name, it, err)
        posted, served, done = bls.bls_counters(plan)
        assert posted == served == done == [it + 1] * P


BULK_CASES = ["cfg1", "cfg3_small", "cfg5_small", "one_rank", "dim128_f32", "extreme_bags", "short_bags_wide_tiles",
              "many_tables", "max_ranks"]


@pytest.mark.parametrize("depth", [16, 32])
@pytest.mark.parametrize("name", BULK_CASES)
def test_bulk_staged_gather_matches_oracle(name, depth):
    """The table-wise gather with rows staged in shared memory by bulk copies (bls_set_tuning,
    16 or 32 rows in flight per lane group): same results as the register path, checked
    against the oracle, over two iterations that reuse the ring's barriers."""
    w = dict(CASES)[name]()
    data = [bi.table_values(t) for t in w.tables]
    tabs = dev_tables(w, data)
    plan = make_plan(w, tabs, k_max=0)
    ref_plan = make_plan(w, tabs, k_max=0)
    bls.bls_set_tuning(plan, 0, depth)
    for it in range(2):
        ids, off = bi.make_iteration(w, it)
        d_ids, d_off = torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda()
        outs = []
        for pl in (plan, ref_plan):
            bls.bls_route(pl, it, d_ids, d_off)
            bls.bls_lookup(pl, it)
            assert bls.bls_status(pl)[0] == bls.BLS_OK
            outs.append(bls.bls_view(pl, it)["out"])
        want = oracle.pool_definition(w.P, w.T, w.local_batch, w.tables, data, ids, off)
        assert oracle.vector_rel_err(outs[0].cpu().numpy(), want) <= TOL[w.tables[0].dtype]
        assert torch.equal(outs[0], outs[1])             # rows are added in the same order: bit-identical


def test_all_bags_empty():
    w = bi.tiny_workload(T=3, P=2, b=4, rows=9, dim=16)
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    plan = make_plan(w, tabs, 0, cap=8)
    off = torch.zeros(2 * 3 * 4 + 1, dtype=torch.int32, device="cuda")
    ids = torch.zeros(0, dtype=torch.int32, device="cuda")
    bls.bls_route(plan, 0, ids, off)
    bls.bls_lookup(plan, 0)
    v = bls.bls_view(plan, 0)
    assert bls.bls_status(plan)[0] == bls.BLS_OK
    assert int(v["sendcounts"].sum()) == 0
    assert torch.count_nonzero(v["out"]).item() == 0


@pytest.mark.parametrize("part", ["table_rr", "row_block"])
def test_bad_inputs_are_reported_not_trapped(part):
    """Out-of-range IDs, a send buffer that is too small and non-monotone offsets
    set the status word; the context stays usable."""
    w = bi.tiny_workload(T=2, P=2, b=3, rows=10, dim=8, partition=part, lengths="one")
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    ids, off = bi.make_iteration(w, 0)
    bad = ids.copy()
    bad[3] = 10
    bad[5] = -1
    plan = make_plan(w, tabs, 0, cap=64)
    bls.bls_route(plan, 0, torch.from_numpy(bad).cuda(), torch.from_numpy(off).cuda())
    bls.bls_lookup(plan, 0)
    assert bls.bls_status(plan)[0] == bls.BLS_ERANGE
    plan = make_plan(w, tabs, 0, cap=2)                       # 6 ids per rank do not fit
    bls.bls_route(plan, 0, torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda())
    bls.bls_lookup(plan, 0)
    assert bls.bls_status(plan)[0] == bls.BLS_ENOSPC
    plan = make_plan(w, tabs, 0, cap=64)
    off2 = off.copy()
    off2[4] = 1
    bls.bls_route(plan, 0, torch.from_numpy(ids).cuda(), torch.from_numpy(off2).cuda())
    bls.bls_lookup(plan, 0)
    assert bls.bls_status(plan)[0] == bls.BLS_EINVAL
    # the device is still healthy
    assert torch.ones(4, device="cuda").sum().item() == 4.0


def test_call_order_is_enforced():
    w = bi.tiny_workload(T=2, P=2, b=3, rows=10, dim=8)
    tabs = dev_tables(w, [bi.table_values(t) for t in w.tables])
    plan = make_plan(w, tabs, 1, cap=64)
    ids, off = bi.make_iteration(w, 0)
    d_ids, d_off = torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda()
    with pytest.raises(bls.BlsError) as e:
        bls.bls_lookup(plan, 0)
    assert e.value.code == bls.BLS_ESTATE
    with pytest.raises(bls.BlsError):
        bls.bls_route(plan, 3, d_ids, d_off)
    with pytest.raises(bls.BlsError):
        bls.bls_step(plan, 2, d_ids, d_off)                   # k > k_max


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_hash_fill_matches_generator(dtype):
    """The device fill kernel and the numpy generator agree bit for bit."""
    w = torch.empty(3000, 64, dtype=TDT[dtype], device="cuda")
    bls.bls_fill_hash_table(w, 4000, 7)
    torch.cuda.synchronize()
    want = bi.hash_rows(4000, 7, np.arange(3000), 64, dtype)
    got = w.cpu()
    got = got.view(torch.int16).numpy().view(np.uint16) if dtype != "f32" else got.numpy()
    want = want.view(np.uint16) if dtype == "f16" else want
    assert np.array_equal(got, want)
