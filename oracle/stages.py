"""CPU oracle of the dense stages either side of the lookup (test infrastructure only).

Listing 1 / Listing 2 of the paper put three dense steps around the embedding exchange:
the bottom MLP on the dense features (it runs between the alltoall and its wait), the
feature interaction of the bottom MLP's output with the pooled embedding vectors, and the
top MLP that turns the interaction into the click probability.  The paper takes these
from the reference DLRM and does not restate them; the definitions below are the usual
ones of that model, written out plainly:

  linear layer   y = act(x W^T + bias)            W [out][in], act = ReLU, or the logistic
                                                  function on the last top layer
  interaction    for one sample, the T + 1 vectors v_0 = bottom output, v_1..v_T = pooled
                 vectors; R = [v_0, <v_i, v_j> for i = 1..T, j = 0..i-1]  (strictly lower
                 triangle, row-major), length D + T (T + 1) / 2

Precision: the CUDA path keeps activations in bfloat16 between layers and accumulates in
fp32.  So that both sides take every rounding decision at the same place, this oracle sums
in fp64 and rounds each layer's output (and the interaction's output) to bfloat16,
round-to-nearest-even, exactly where the CUDA path stores bfloat16; the final probability
is rounded to fp32.  Nothing here shares code with the CUDA library.

Pins (tests/test_oracle_stages.py): nested Python loops on tiny cases, identity weights,
torch.nn.functional.linear and torch.bmm in fp64, the closed form of the logistic function.
No function here is "parity unpinned".
"""
from __future__ import annotations

from typing import Sequence

import numpy as np


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp64/fp32 values to the nearest bfloat16 (ties to even), returned as float64."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)      # one rounding to fp32 first, as a conversion chain would
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = (u + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def linear(x: np.ndarray, weight: np.ndarray, bias: np.ndarray, act: str) -> np.ndarray:
    """y = act(x W^T + bias) in fp64.  x [rows][in], weight [out][in], bias [out]."""
    y = np.asarray(x, np.float64) @ np.asarray(weight, np.float64).T + np.asarray(bias, np.float64)
    if act == "relu":
        return np.maximum(y, 0.0)
    if act == "sigmoid":
        return 1.0 / (1.0 + np.exp(-y))
    if act == "none":
        return y
    raise ValueError(act)


def mlp(x: np.ndarray, weights: Sequence[np.ndarray], biases: Sequence[np.ndarray], last_act: str) -> np.ndarray:
    """ReLU layers, the last one with `last_act`; every layer's output except the last is
    rounded to bfloat16, the last one to bfloat16 when last_act is "relu" (it feeds the
    interaction) and to fp32 otherwise (the click probability)."""
    h = np.asarray(x, np.float64)
    n = len(weights)
    for i, (w, b) in enumerate(zip(weights, biases)):
        last = i == n - 1
        h = linear(h, w, b, last_act if last else "relu")
        h = h.astype(np.float32).astype(np.float64) if (last and last_act != "relu") else round_bf16(h)
    return h


def interact(x: np.ndarray, pooled: np.ndarray) -> np.ndarray:
    """x [B][D] (bottom output), pooled [B][T][D] -> R [B][D + T(T+1)/2], rounded to bfloat16."""
    x = np.asarray(x, np.float64)
    pooled = np.asarray(pooled, np.float64)
    B, T, D = pooled.shape
    v = np.concatenate([x.reshape(B, 1, D), pooled], axis=1)                # [B][T+1][D]
    out = np.zeros((B, D + T * (T + 1) // 2), np.float64)
    out[:, :D] = x
    c = D
    for i in range(1, T + 1):
        for j in range(i):
            out[:, c] = np.sum(v[:, i, :] * v[:, j, :], axis=1)
            c += 1
    return round_bf16(out)


def forward(dense_x, pooled, bot_w, bot_b, top_w, top_b) -> np.ndarray:
    """Click probability per sample: bottom MLP -> interaction with the pooled vectors -> top MLP."""
    x = mlp(dense_x, bot_w, bot_b, "relu")
    r = interact(x, pooled)
    pad = top_w[0].shape[1] - r.shape[1]                                    # the first top layer may be zero-padded on its input side
    if pad > 0:
        r = np.concatenate([r, np.zeros((r.shape[0], pad))], axis=1)
    return mlp(r, top_w, top_b, "sigmoid")
