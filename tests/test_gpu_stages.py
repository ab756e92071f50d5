"""The dense stages either side of the lookup (bottom MLP, feature interaction, top MLP;
Listing 1 / Listing 2) on the GPU - tensor-core linear layers and the interaction kernel -
against the fp64 oracle of oracle/stages.py, through the C ABI.  GPU only.

Tolerance: both sides round activations to bfloat16 at the same places; the CUDA path sums
in fp32, the oracle in fp64, so a sum that lands within fp32 round-off of a bfloat16 tie can
round the other way (one unit in the last place, 2^-8 relative) and that difference travels
on through the following layers.  Bar: per output vector max|g - o| / max|o| <= 1e-2 (the
bar for bf16 data), and 2e-3 absolute on the final probability."""
import numpy as np
import pytest
import torch

import bls_inputs as bi
import oracle
import paper_2512_19342_b200 as bls
from oracle import stages

pytestmark = pytest.mark.gpu


def bf16_values(rng, shape, scale):
    """Random values that are exactly representable in bfloat16 (as float64 array)."""
    return stages.round_bf16(rng.standard_normal(shape) * scale)


def to_dev_bf16(a):
    return torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16).cuda().contiguous()


def make_mlp(rng, dims, last_act, max_rows):
    ws = [bf16_values(rng, (dims[i + 1], dims[i]), 1.0 / np.sqrt(dims[i])) for i in range(len(dims) - 1)]
    bs = [rng.standard_normal(dims[i + 1]).astype(np.float32).astype(np.float64) * 0.1 for i in range(len(dims) - 1)]
    mlp = bls.Mlp([to_dev_bf16(w) for w in ws], [torch.from_numpy(b.astype(np.float32)).cuda() for b in bs], last_act, max_rows)
    return mlp, ws, bs


@pytest.mark.parametrize("rows,dims,last_act", [
    (128, [64, 128], 1),                       # one tile, one K block
    (300, [16, 512, 256, 64], 1),              # bottom MLP shape: ragged rows, K = 16 (zero-filled to 64), several N tiles
    (1000, [448, 512, 256, 8], 2),             # top MLP shape: 7 K blocks (the ring wraps), narrow last layer, logistic output
    (77, [200, 96, 40], 0),                    # K, N not multiples of the tile sizes
    (2048, [64, 64, 64, 64, 64], 1),           # many layers on one handle
])
def test_mlp_matches_oracle(rows, dims, last_act):
    rng = np.random.Generator(np.random.PCG64(sum(dims) + rows))
    mlp, ws, bs = make_mlp(rng, dims, last_act, max_rows=rows + 5)
    x = bf16_values(rng, (rows, dims[0]), 1.0)
    act = {0: "none", 1: "relu", 2: "sigmoid"}[last_act]
    for y_dtype in ((torch.bfloat16,) if last_act == 1 else (torch.float32,)):
        y = torch.full((rows, dims[-1]), float("nan"), dtype=y_dtype, device="cuda")
        for _ in range(2):                                     # twice: barriers and tensor memory are set up per launch
            mlp.forward(to_dev_bf16(x), y)
        assert mlp.status() == bls.BLS_OK
        want = stages.mlp(x, ws, bs, act)
        got = y.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        assert oracle.vector_rel_err(got, want) <= 1e-2
    if last_act == 2:
        assert np.abs(got - want).max() <= 2e-3


def test_linear_layer_with_identity_weights_copies_relu_of_input():
    """Exact case: W = I, bias = 0 -> y = relu(x) bit for bit (every product is x * 1, every sum has one term)."""
    rng = np.random.Generator(np.random.PCG64(9))
    n, rows = 128, 260
    x = bf16_values(rng, (rows, n), 2.0)
    mlp = bls.Mlp([to_dev_bf16(np.eye(n))], [torch.zeros(n, device="cuda")], 1, rows)
    y = torch.empty(rows, n, dtype=torch.bfloat16, device="cuda")
    mlp.forward(to_dev_bf16(x), y)
    assert mlp.status() == bls.BLS_OK
    assert np.array_equal(y.float().cpu().numpy().astype(np.float64), np.maximum(x, 0.0))
    # a permutation matrix shows that no operand is transposed and no tile is misplaced
    perm = rng.permutation(n)
    pm = np.zeros((n, n))
    pm[np.arange(n), perm] = 1.0                              # y[:, o] = x[:, perm[o]]
    mlp = bls.Mlp([to_dev_bf16(pm)], [torch.zeros(n, device="cuda")], 0, rows)
    y32 = torch.empty(rows, n, dtype=torch.float32, device="cuda")
    mlp.forward(to_dev_bf16(x), y32)
    assert np.array_equal(y32.cpu().numpy().astype(np.float64), x[:, perm])


@pytest.mark.parametrize("B,T,D", [(64, 26, 64), (33, 3, 16), (5, 8, 128)])
def test_interaction_matches_oracle(B, T, D):
    rng = np.random.Generator(np.random.PCG64(B + T + D))
    x = bf16_values(rng, (B, D), 1.0)
    pooled = (rng.standard_normal((B, T, D)) * 2.0).astype(np.float32)
    n_out = D + T * (T + 1) // 2
    ldr = (n_out + 63) // 64 * 64
    r = torch.full((B, ldr), float("nan"), dtype=torch.bfloat16, device="cuda")
    bls.bls_interact(to_dev_bf16(x), torch.from_numpy(pooled).cuda(), r)
    torch.cuda.synchronize()
    got = r.float().cpu().numpy().astype(np.float64)
    want = stages.interact(x, pooled)
    assert np.array_equal(got[:, :D], x)                       # the bottom output is copied through
    assert np.all(got[:, n_out:] == 0)                         # padding
    assert oracle.vector_rel_err(got[:, :n_out], want) <= 1e-2


def test_lookup_and_stages_end_to_end():
    """bottom MLP -> BLS lookup (k = 1) -> interaction -> top MLP on the GPU against the oracle chain
    (oracle pooling by definition, then oracle/stages.forward)."""
    w = bi.workload(3, 0.01, 0.02)                              # 26 tables, P = 8, D = 64
    data = [bi.table_values(t) for t in w.tables]
    tabs = [torch.from_numpy(d).cuda() for d in data]
    P, T, b, D = w.P, w.T, w.local_batch, w.tables[0].dim
    B = P * b
    rng = np.random.Generator(np.random.PCG64(77))
    bot, bw, bb = make_mlp(rng, [16, 128, D], 1, B)
    n_int = D + T * (T + 1) // 2
    ldr = (n_int + 63) // 64 * 64
    # 8 outputs; no logistic function at the end here: with N(0,1) table rows the pooled vectors are large and the
    # probabilities saturate at 0 or 1, which would hide errors, so the test compares the logits
    top, tw, tb = make_mlp(rng, [ldr, 256, 64, 8], 0, B)
    inputs = [bi.make_iteration(w, t) for t in range(3)]
    dense = [bf16_values(rng, (B, 16), 1.0) for _ in inputs]
    cap = max(int(np.diff(off[::T * b].astype(np.int64)).max()) for _, off in inputs) + 16
    plan = bls.bls_plan(tabs, w.partition, P, b, 1, cap)
    xs, got = {}, {}
    r = torch.empty(B, ldr, dtype=torch.bfloat16, device="cuda")

    def finish(out, it):
        bls.bls_interact(xs[it], out, r)
        p = torch.empty(B, 8, dtype=torch.float32, device="cuda")
        top.forward(r, p)
        got[it] = p.cpu().numpy()

    for t, (ids, off) in enumerate(inputs):
        out, it = bls.bls_step(plan, 1, torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda())
        xs[t] = torch.empty(B, D, dtype=torch.bfloat16, device="cuda")
        bot.forward(to_dev_bf16(dense[t]), xs[t])               # the bottom MLP of batch t runs while its lookup is in flight
        if out is not None:
            finish(out, it)
    while True:
        out, it = bls.bls_drain(plan)
        if out is None:
            break
        finish(out, it)
    assert bls.bls_status(plan)[0] == bls.BLS_OK and bot.status() == bls.BLS_OK and top.status() == bls.BLS_OK
    for t, (ids, off) in enumerate(inputs):
        pooled = oracle.pool_definition(P, T, b, w.tables, data, ids, off).reshape(B, T, D)
        x = stages.mlp(dense[t], bw, bb, "relu")
        r_want = np.concatenate([stages.interact(x, pooled), np.zeros((B, ldr - n_int))], axis=1)
        want = stages.mlp(r_want, tw, tb, "none")
        err = oracle.vector_rel_err(got[t].astype(np.float64), want)
        assert err <= 1e-2, (t, err)


def test_stage_calls_reject_bad_arguments():
    """Argument checks of the dense-stage entry points happen on the host, before any GPU work."""
    import ctypes as C
    lib = bls.lib()
    n = C.c_size_t(0)
    dims = (C.c_int * 3)(16, 12, 8)                          # a hidden width that is not a multiple of 8
    assert lib.bls_mlp_bytes(2, dims, 128, C.byref(n)) == bls.BLS_EINVAL
    dims = (C.c_int * 3)(16, 64, 8)
    assert lib.bls_mlp_bytes(2, dims, 0, C.byref(n)) == bls.BLS_EINVAL
    assert lib.bls_mlp_bytes(2, dims, 128, C.byref(n)) == bls.BLS_OK and n.value >= 128 * 64 * 2
    rng = np.random.Generator(np.random.PCG64(0))
    mlp, _, _ = make_mlp(rng, [16, 64, 8], 1, 128)
    x = torch.zeros(200, 16, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(200, 8, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bls.BlsError) as e:
        mlp.forward(x, y)                                    # more rows than the handle was made for
    assert e.value.code == bls.BLS_EINVAL
    with pytest.raises(bls.BlsError):
        bls.bls_interact(x, torch.zeros(200, 3, 16, device="cuda"), torch.zeros(200, 16, dtype=torch.bfloat16, device="cuda"))   # r too narrow
    assert torch.ones(4, device="cuda").sum().item() == 4.0
