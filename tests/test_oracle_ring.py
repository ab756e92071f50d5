"""Pins for the slot-ring model (bounded lag), CPU only."""
import numpy as np
import pytest

from oracle.ring_model import RingModel, makespan


@pytest.mark.parametrize("k", [0, 1, 2, 4, 8])
@pytest.mark.parametrize("P", [1, 3, 8])
def test_random_legal_schedules(P, k):
    """Any legal interleaving completes every iteration, in order, within the bound."""
    n = 12
    for seed in range(5):
        m = RingModel(P, k, n).run_random(seed * 101 + P * 7 + k)
        # drain: everything issued was completed (Listing 2's final loop)
        assert sorted(m.completed) == [(r, j) for r in range(P) for j in range(n)]
        # FIFO: a rank completes its requests oldest first (Section III-B, wait())
        for r in range(P):
            assert [j for rr, j in m.completed if rr == r] == list(range(n))
        # bounded lag (Section I: |j - i| <= k)
        assert m.max_spread <= k
        # output sequence identical to the synchronous one (k = 0 has a single order per rank)
        ref = RingModel(P, 0, n).run_random(0)
        for r in range(P):
            assert [j for rr, j in m.completed if rr == r] == [j for rr, j in ref.completed if rr == r]


def test_k0_is_lockstep():
    """Bound 0: nobody posts iteration j+1 before everyone has completed j."""
    m = RingModel(4, 0, 6).run_random(3)
    posted_at = {}
    done_at = {}
    for i, (kind, r, j) in enumerate(m.trace):
        if kind == "post":
            posted_at[(r, j)] = i
        if kind == "consume":
            done_at[(r, j)] = i
    for j in range(5):
        assert min(posted_at[(r, j + 1)] for r in range(4)) > max(done_at[(r, j)] for r in range(4))


def test_bound_figure_scenario():
    """Section III-D's figure: three ranks in iterations 0, 2 and 1, three buffers.
    The leader has sent iterations 0..2, cannot complete iteration 0 before the
    slowest rank has sent it, and may reuse that buffer for iteration 3 only after."""
    m = RingModel(3, 2, 6)
    for _ in range(3):
        m.post(1)                       # P1 sent iterations 0, 1, 2
    for _ in range(2):
        m.post(2)                       # P2 sent iterations 0, 1
    assert not m.can_post(1)            # buffer 0 still holds iteration 0
    assert not m.can_consume(1)         # P0's data for iteration 0 has not arrived
    assert not any(m.can_serve(o) for o in range(3))
    m.post(0)                           # P0 sends iteration 0
    for o in range(3):
        m.serve(o)
    assert m.can_consume(1)
    m.consume(1)
    assert not m.can_post(1)            # the buffer is shared: every rank must have read it
    m.consume(0)
    m.consume(2)
    assert m.can_post(1)
    m.post(1)
    assert ("post", 1, 3) == m.trace[-1] and 3 % m.S == 0   # iteration 3 reuses buffer 0


def test_planted_mistake_missing_gate_is_caught():
    """Without the consumer-progress gate a fast rank overwrites unread data: the
    model's poison check must fire.  (The mistake is planted in the model, on the CPU.)"""
    class NoGate(RingModel):
        def can_post(self, r):
            return self.posted[r] < self.n_iter
    m = NoGate(2, 1, 6)
    with pytest.raises(AssertionError):
        for _ in range(3):
            m.post(0)


def test_ring_memory_closed_form():
    """Section V-F: one alltoallv buffer holds s*b*|tables| bytes, independent of
    table sizes; b=512, s=64 B, 26 tables is about 860 KB per unit of k."""
    assert 64 * 512 * 26 == 851_968
    assert abs(851_968 / 1000 - 860) < 10


def test_delay_masking_closed_forms():
    """Section VI-B: uniform random delays U(0, 2d) per step are masked for k > 0,
    with gains that diminish quickly as k grows.  Synchronous: every iteration
    costs the maximum delay over the P ranks, E = 2d*P/(P+1).  Unbounded: each
    rank runs at its own mean d."""
    rng = np.random.Generator(np.random.PCG64(5))
    P, n, d = 8, 1500, 0.005
    delays = rng.uniform(0, 2 * d, size=(P, n))
    ts = {k: makespan(delays, k) / n for k in (0, 1, 2, 4, 8, n)}
    assert abs(ts[0] - 2 * d * P / (P + 1)) < 2e-4
    assert abs(ts[n] - d) < 3e-4
    ks = sorted(ts)
    assert all(ts[a] >= ts[b] - 1e-12 for a, b in zip(ks, ks[1:]))      # monotone in k
    assert ts[0] - ts[1] > 0.5 * (ts[0] - ts[n])                        # most of the gain at k = 1
    assert ts[8] - ts[n] < 0.1 * (ts[0] - ts[n])                        # and little left after k = 8


def test_constant_straggler_is_not_masked():
    """Section IV, last paragraph: one consistently slow rank cannot be hidden."""
    P, n = 8, 500
    delays = np.zeros((P, n))
    delays[3] = 0.01
    for k in (0, 1, 4, 8):
        assert abs(makespan(delays, k) / n - 0.01) < 1e-3
