"""Pins of the dense-stage oracle (oracle/stages.py): each function against something
other than itself - nested loops, identity weights, library routines, closed forms."""
import numpy as np
import torch

from oracle import stages


def test_round_bf16_matches_torch_on_every_interesting_pattern():
    rng = np.random.Generator(np.random.PCG64(5))
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-6, 6, 20000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.0 + 2.0 ** -9, 1.0 + 3 * 2.0 ** -9, 65504.0, 3.0e38]])
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(stages.round_bf16(x), want)
    # ties go to the even neighbour: 1 + 2^-8 lies exactly between 1 and 1 + 2^-7
    assert stages.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert stages.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6


def test_linear_brute_force_and_library():
    rng = np.random.Generator(np.random.PCG64(1))
    x, w, b = rng.standard_normal((5, 7)), rng.standard_normal((3, 7)), rng.standard_normal(3)
    want = np.zeros((5, 3))
    for r in range(5):
        for o in range(3):
            s = b[o]
            for i in range(7):
                s += x[r, i] * w[o, i]                   # W is [out][in]: a transposed operand would fail here
            want[r, o] = max(s, 0.0)
    assert np.allclose(stages.linear(x, w, b, "relu"), want, rtol=0, atol=1e-12)
    lib = torch.nn.functional.linear(torch.from_numpy(x), torch.from_numpy(w), torch.from_numpy(b))
    assert np.allclose(stages.linear(x, w, b, "none"), lib.numpy(), rtol=0, atol=1e-12)
    assert np.allclose(stages.linear(x, w, b, "sigmoid"), torch.sigmoid(lib).numpy(), rtol=0, atol=1e-12)
    # logistic function: closed forms
    assert stages.linear(np.zeros((1, 7)), w, np.zeros(3), "sigmoid")[0, 0] == 0.5
    assert abs(stages.linear(np.zeros((1, 7)), w, np.full(3, np.log(3.0)), "sigmoid")[0, 0] - 0.75) < 1e-15


def test_mlp_with_identity_weights_is_relu_of_the_rounded_input():
    x = np.array([[1.0, -2.0, 0.5, 3.0], [0.25, 0.0, -1.0, 1.0 + 2.0 ** -10]])
    eye, zero = np.eye(4), np.zeros(4)
    got = stages.mlp(x, [eye, eye], [zero, zero], "relu")
    assert np.array_equal(got, stages.round_bf16(np.maximum(x, 0.0)))
    # a bias only on the second layer shows that layers are applied in order
    got = stages.mlp(x, [eye, eye], [zero, np.array([1.0, 0, 0, 0])], "relu")
    assert got[0, 0] == 2.0 and got[0, 1] == 0.0
    # the last layer of a top MLP is not rounded to bfloat16
    p = stages.mlp(np.array([[0.3]]), [np.array([[1.0]])], [np.zeros(1)], "sigmoid")[0, 0]
    assert p == np.float32(1.0 / (1.0 + np.exp(-0.3)))


def test_interact_against_loops_and_bmm():
    rng = np.random.Generator(np.random.PCG64(2))
    B, T, D = 4, 5, 8
    x = stages.round_bf16(rng.standard_normal((B, D)))
    pooled = rng.standard_normal((B, T, D)).astype(np.float32).astype(np.float64)
    got = stages.interact(x, pooled)
    assert got.shape == (B, D + T * (T + 1) // 2)
    for b in range(B):
        v = [x[b]] + [pooled[b, t] for t in range(T)]
        want = list(x[b])
        for i in range(1, T + 1):
            for j in range(i):
                want.append(sum(v[i][c] * v[j][c] for c in range(D)))
        assert np.array_equal(got[b], stages.round_bf16(np.array(want)))
    # library route: all pairwise products by a batched matrix product, strictly lower triangle row by row
    v = torch.from_numpy(np.concatenate([x.reshape(B, 1, D), pooled], axis=1))
    z = torch.bmm(v, v.transpose(1, 2)).numpy()
    li, lj = np.tril_indices(T + 1, -1)
    assert np.allclose(got[:, D:], stages.round_bf16(z[:, li, lj]), rtol=2.0 ** -7, atol=1e-12)
    # identifying input: one-hot vectors make <v_i, v_j> = 1 only for the pair that shares a coordinate
    one = np.zeros((1, 3, 4))
    one[0, 0, 1] = 1.0
    one[0, 2, 1] = 1.0                                    # v_1 and v_3 share coordinate 1
    r = stages.interact(np.zeros((1, 4)), one)[0, 4:]
    pairs = [(i, j) for i in range(1, 4) for j in range(i)]
    assert [pairs[q] for q in np.nonzero(r)[0]] == [(3, 1)]


def test_forward_chains_the_three_stages():
    rng = np.random.Generator(np.random.PCG64(3))
    B, T, D = 3, 2, 8
    dense = stages.round_bf16(rng.standard_normal((B, 8)))
    pooled = rng.standard_normal((B, T, D)).astype(np.float32)
    bw = [stages.round_bf16(rng.standard_normal((16, 8)) * 0.3), stages.round_bf16(rng.standard_normal((D, 16)) * 0.3)]
    bb = [rng.standard_normal(16) * 0.1, rng.standard_normal(D) * 0.1]
    n_in = D + T * (T + 1) // 2
    tw = [stages.round_bf16(rng.standard_normal((8, 16)) * 0.3), stages.round_bf16(rng.standard_normal((1, 8)) * 0.3)]
    tb = [rng.standard_normal(8) * 0.1, rng.standard_normal(1) * 0.1]
    assert n_in == 11                                     # the first top layer is zero-padded from 11 to 16 inputs
    p = stages.forward(dense, pooled, bw, bb, tw, tb)
    x = stages.mlp(dense, bw, bb, "relu")
    r = np.concatenate([stages.interact(x, pooled), np.zeros((B, 5))], axis=1)
    assert np.array_equal(p, stages.mlp(r, tw, tb, "sigmoid"))
    assert p.shape == (B, 1) and np.all((p > 0) & (p < 1))
