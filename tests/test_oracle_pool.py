"""Pins for the oracle's pooled output (steps 2 and 3) and its value decoders, CPU only."""
import numpy as np
import pytest
import torch

import bls_inputs as bi
import oracle


def _setup(w, it=0):
    ids, off = bi.make_iteration(w, it)
    data = [bi.table_values(t) for t in w.tables]
    return ids, off, data


def _rows(w):
    return [t.rows for t in w.tables]


def test_brute_force_python_loops():
    """Tiny input, the definition written as nested Python loops over dicts."""
    w = bi.tiny_workload(T=3, P=2, b=2, rows=[4, 6, 5], dim=2)
    ids, off = bi.make_iteration(w, 0)
    data = [np.array([[100.0 * t + r + 0.25 * c for c in range(2)] for r in range(tb.rows)], np.float32)
            for t, tb in enumerate(w.tables)]
    got = oracle.pool_definition(2, 3, 2, w.tables, data, ids, off)
    for src in range(2):
        for t in range(3):
            for s in range(2):
                g = (src * 3 + t) * 2 + s
                want = [0.0, 0.0]
                for l in range(off[g], off[g + 1]):
                    for c in range(2):
                        want[c] += 100.0 * t + int(ids[l]) + 0.25 * c
                assert got[src, s, t].tolist() == want


@pytest.mark.parametrize("part", ["table_rr", "row_block"])
def test_all_ones_table_gives_bag_length(part):
    w = bi.tiny_workload(T=5, P=4, b=6, rows=37, dim=8, partition=part, lengths="poisson10")
    ids, off = bi.make_iteration(w, 0)
    data = [np.ones((37, 8), np.float32)] * 5
    lens = np.diff(off).reshape(4, 5, 6).transpose(0, 2, 1)          # [src][s][t]
    d = oracle.pool_definition(4, 5, 6, w.tables, data, ids, off)
    assert np.array_equal(d, np.broadcast_to(lens[..., None], d.shape).astype(np.float32))
    art = oracle.route(4, 5, 6, part, _rows(w), ids, off)
    r = oracle.pool_routed(4, 5, 6, part, w.tables, data, art)
    assert np.array_equal(r, d)


@pytest.mark.parametrize("part", ["table_rr", "row_block"])
def test_identifying_table_pins_return_layout(part):
    """One-hot lookups into W_t[id][c] = t*2^20 + id + c*2^-3: every output element
    names its table, row and column exactly, so any misplacement is a mismatch."""
    w = bi.tiny_workload(T=6, P=3, b=5, rows=1000, dim=4, partition=part, lengths="one")
    ids, off = bi.make_iteration(w, 2)
    data = [(t * 2 ** 20 + np.arange(1000)[:, None] + np.arange(4)[None, :] / 8.0).astype(np.float32)
            for t in range(6)]
    art = oracle.route(3, 6, 5, part, _rows(w), ids, off)
    for out in (oracle.pool_definition(3, 6, 5, w.tables, data, ids, off),
                oracle.pool_routed(3, 6, 5, part, w.tables, data, art)):
        idm = ids.reshape(3, 6, 5).transpose(0, 2, 1)                   # [src][s][t]
        want = (np.arange(6)[None, None, :] * 2 ** 20 + idm)[..., None] + np.arange(4) / 8.0
        assert np.array_equal(out, want.astype(np.float32))


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_single_rank_equals_embedding_bag(dtype):
    """P = 1, one table: the path is a plain embedding-bag sum (Listing 1's apply_emb)."""
    w = bi.tiny_workload(T=1, P=1, b=200, rows=500, dim=16, dtype=dtype, lengths="poisson20c")
    ids, off, data = _setup(w)
    if dtype == "f32":
        W = torch.from_numpy(data[0]).double()
    elif dtype == "f16":
        W = torch.from_numpy(data[0]).double()
    else:
        W = torch.from_numpy(data[0].view(np.int16)).view(torch.bfloat16).double()
    ref = torch.nn.functional.embedding_bag(torch.from_numpy(ids).long(), W,
                                            torch.from_numpy(off[:-1]).long(), mode="sum")
    got = oracle.pool_definition(1, 1, 200, w.tables, data, ids, off).reshape(200, 16)
    np.testing.assert_allclose(got, ref.numpy().astype(np.float32), rtol=2e-7, atol=0)


@pytest.mark.parametrize("num,rs,bs", [(1, 1.0, 1.0), (3, 0.002, 0.01), (4, 0.0005, 0.002), (5, 0.0002, 0.001)])
def test_definition_equals_routed_evaluation(num, rs, bs):
    """The route must be a bag-preserving permutation: pooling what the owners
    received gives the same result as pooling the original bags."""
    w = bi.workload(num, rs, bs)
    ids, off, data = _setup(w)
    P, T, b = w.P, w.T, w.local_batch
    d = oracle.pool_definition(P, T, b, w.tables, data, ids, off)
    art = oracle.route(P, T, b, w.partition, _rows(w), ids, off)
    r = oracle.pool_routed(P, T, b, w.partition, w.tables, data, art)
    if w.partition == "table_rr":
        assert np.array_equal(d, r)                 # same addends in the same order
    else:
        np.testing.assert_allclose(r, d, rtol=1e-6, atol=1e-6)   # owner order regroups the sum
    # and evaluating the hash on demand equals reading the materialised table
    if w.tables[0].kind == "hash":
        d2 = oracle.pool_definition(P, T, b, w.tables, None, ids, off)
        assert np.array_equal(d, d2)


def test_selected_bags_match_full_evaluation():
    w = bi.workload(3, 0.002, 0.01)
    ids, off, data = _setup(w)
    P, T, b = w.P, w.T, w.local_batch
    full = oracle.pool_definition(P, T, b, w.tables, data, ids, off)
    sel = np.array([0, 7, P * T * b - 1, 123], np.int64)
    part = oracle.pool_definition(P, T, b, w.tables, None, ids, off, sel=sel)
    for i, g in enumerate(sel):
        src, t, s = g // (T * b), (g // b) % T, g % b
        assert np.array_equal(part[i], full[src, s, t])


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_hash_fill_two_independent_implementations(dtype):
    """The C oracle and the numpy generator implement the same published
    counter generator and rounding rules; they must agree bit for bit.  With
    about 1e6 values this also exercises fp16 subnormals and ties."""
    spec = bi.TableSpec(rows=16384, dim=64, dtype=dtype, kind="hash", seed=4000, index=5)
    a = oracle.fill_table(spec, nthreads=4)
    b = bi.hash_rows(spec.seed, spec.index, np.arange(spec.rows), spec.dim, dtype)
    if dtype == "f16":
        b = b.view(np.uint16)
    assert np.array_equal(a, b)
    v = bi.hash_rows(spec.seed, spec.index, np.arange(spec.rows), spec.dim, "f32")
    assert abs(float(v.mean())) < 0.01 and abs(float(v.std()) - 1.0) < 0.01


def test_low_precision_decoders_against_libraries():
    """All 65536 bit patterns: fp16 vs numpy's float16, bf16 vs torch's bfloat16."""
    bits = np.arange(65536, dtype=np.uint16).reshape(-1, 1)
    for dtype, ref in (("f16", bits.view(np.float16).astype(np.float64)),
                       ("bf16", torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).double().numpy())):
        spec = bi.TableSpec(rows=65536, dim=1, dtype=dtype, kind="normal", seed=0, index=0)
        ids = np.arange(65536, dtype=np.int32)
        off = np.arange(65537, dtype=np.int32)
        got = oracle.pool_definition(1, 1, 65536, [spec], [bits], ids, off).reshape(-1)
        want = ref.reshape(-1).astype(np.float32)
        ok = np.isfinite(want)
        assert np.array_equal(got[ok], want[ok])
        assert np.all(np.isnan(got[np.isnan(want)]))
        assert np.array_equal(got[np.isinf(want)], want[np.isinf(want)])


def test_fp32_summation_error_is_far_inside_tolerance():
    """The only rounding on the GPU side is fp32 accumulation order.  For bags of
    at most 100 values the forward error bound len * 2^-24 * sum|w| stays far below
    the 1e-5 bar relative to sum|w|; check it on the worst bag length."""
    rng = np.random.Generator(np.random.PCG64(11))
    w = rng.standard_normal((100, 64)).astype(np.float32)
    exact = w.astype(np.float64).sum(0)
    f32 = np.zeros(64, np.float32)
    for r in w:
        f32 = f32 + r
    assert np.all(np.abs(f32 - exact) <= 100 * 2.0 ** -24 * np.abs(w).sum(0))
    assert np.abs(f32 - exact).max() / np.abs(exact).max() < 1e-5
