"""Discrete-event model of the bounded-lag-synchronous slot ring (test infrastructure).

P ranks exchange one request message and one response message per iteration.
Iteration j lives in slot j mod (k+1).  Three monotone counters per rank record
progress (Section III-C: tagged puts are counted per iteration; Section IV,
Listing 2: a rank may run ahead until more than k requests are outstanding, completion is FIFO,
and the last batch drains everything):

  posted[r]  iterations whose requests rank r has put into all owners' slots
  served[o]  iterations owner o has answered into all requesters' slots
  done[r]    iterations rank r has completed (oldest first)

Enabling rules (reading of Section III-D and Listing 2's comment that a rank too
far ahead would overwrite a buffer that is still in use):
  post(r, j)    needs min over ranks of done >= j - k      (slot j mod S is free)
  serve(o, j)   needs every rank to have posted j          (all P sources, self included)
  consume(r, j) needs every owner to have served j         (all P messages with that tag)

``RingModel`` executes any legal interleaving and checks that no slot is read
before it is written or overwritten before it is read (freed entries are
poisoned).  ``makespan`` evaluates the timing recursion of Listing 2 for given
per-(rank, iteration) delays.
"""
from __future__ import annotations

import numpy as np

POISON = -1


class RingModel:
    def __init__(self, P: int, k: int, n_iter: int):
        self.P, self.k, self.S, self.n_iter = P, k, k + 1, n_iter
        self.posted = [0] * P
        self.served = [0] * P
        self.done = [0] * P
        # request[o][slot][src] and response[r][slot][o] hold the iteration tag or POISON
        self.request = [[[POISON] * P for _ in range(self.S)] for _ in range(P)]
        self.response = [[[POISON] * P for _ in range(self.S)] for _ in range(P)]
        self.completed = []            # (rank, iteration) in completion order
        self.max_spread = 0
        self.trace = []

    # -- enabling -----------------------------------------------------------
    def can_post(self, r):
        j = self.posted[r]
        return j < self.n_iter and min(self.done) >= j - self.k

    def can_serve(self, o):
        j = self.served[o]
        return j < self.n_iter and min(self.posted) > j

    def can_consume(self, r):
        j = self.done[r]
        return j < self.n_iter and min(self.served) > j

    def enabled(self):
        acts = []
        for r in range(self.P):
            if self.can_post(r):
                acts.append(("post", r))
            if self.can_serve(r):
                acts.append(("serve", r))
            if self.can_consume(r):
                acts.append(("consume", r))
        return acts

    # -- effects ------------------------------------------------------------
    def post(self, r):
        assert self.can_post(r)
        j = self.posted[r]
        s = j % self.S
        for o in range(self.P):
            assert self.request[o][s][r] == POISON, "request slot overwritten before it was served"
            self.request[o][s][r] = j
        self.posted[r] = j + 1
        self._note(("post", r, j))

    def serve(self, o):
        assert self.can_serve(o)
        j = self.served[o]
        s = j % self.S
        for src in range(self.P):
            assert self.request[o][s][src] == j, "owner read a request of another iteration"
            self.request[o][s][src] = POISON
            assert self.response[src][s][o] == POISON, "response slot overwritten before it was consumed"
            self.response[src][s][o] = j
        self.served[o] = j + 1
        self._note(("serve", o, j))

    def consume(self, r):
        assert self.can_consume(r)
        j = self.done[r]
        s = j % self.S
        for o in range(self.P):
            assert self.response[r][s][o] == j, "requester read a response of another iteration"
            self.response[r][s][o] = POISON
        self.done[r] = j + 1
        self.completed.append((r, j))
        self._note(("consume", r, j))

    def _note(self, ev):
        self.trace.append(ev)
        # Section III (definition of the bound k): the iterations two ranks are
        # working on never differ by more than k.  The fastest rank is inside the
        # newest iteration it has posted, the slowest is still inside the oldest
        # iteration not yet completed.
        self.max_spread = max(self.max_spread, max(self.posted) - 1 - min(self.done))

    def finished(self):
        return all(d == self.n_iter for d in self.done)

    def run_random(self, seed: int):
        rng = np.random.Generator(np.random.PCG64(seed))
        while not self.finished():
            acts = self.enabled()
            assert acts, "deadlock: no enabled action"
            kind, r = acts[int(rng.integers(len(acts)))]
            getattr(self, kind)(r)
        return self


def makespan(delays: np.ndarray, k: int, work: float = 0.0, tail: float = 0.0) -> float:
    """Completion time of a BLS inference loop under per-(rank, iteration) delays.

    Each rank runs the loop of Listing 2: in iteration j it spends
    delay[r][j] + work, issues its exchange for j (not before every rank has
    completed iteration j-k-1, whose buffer it reuses), then completes, oldest
    first, every outstanding request whose data has already arrived; while more
    than k requests are outstanding it blocks on the oldest one.  A request of
    iteration i has arrived once every rank has issued i.  Each completion costs
    ``tail``.  After the last iteration the outstanding requests drain in order.
    Returns the time at which the last rank finishes.

    (Completing requests as soon as they have arrived, rather than only when the
    bound forces it, is what lets a buffer be reused early; with the explicit
    reuse gate above, completing only under pressure would tie every rank to the
    slowest one again.)
    """
    P, n = delays.shape
    INF = float("inf")
    issued = np.full((P, n), INF)
    compl = np.full((P, n), INF)
    now = np.zeros(P)
    nxt = [0] * P                      # next iteration to issue
    done = [0] * P                     # requests completed
    stalled = [False] * P              # delay of iteration nxt already spent

    def arrived(i):                    # time request i is complete everywhere (INF if not yet known)
        return issued[:, i].max()

    def step(r):
        # 1. complete what must or can be completed
        if done[r] < nxt[r]:
            i = done[r]
            a = arrived(i)
            must = (nxt[r] - done[r] > k) or nxt[r] == n
            if a <= now[r] or (must and a < INF):
                now[r] = max(now[r], a) + tail
                compl[r, i] = now[r]
                done[r] += 1
                return True
            if must:
                return False           # blocked on a request that has not arrived
        # 2. issue the next iteration
        if nxt[r] < n:
            j = nxt[r]
            if not stalled[r]:
                now[r] += delays[r, j] + work
                stalled[r] = True
                return True
            if j - k - 1 >= 0:
                free = compl[:, j - k - 1].max()
                if free == INF:
                    return False       # buffer still in use somewhere
                now[r] = max(now[r], free)
            issued[r, j] = now[r]
            nxt[r] += 1
            stalled[r] = False
            return True
        return False

    while any(d < n for d in done):
        for r in np.argsort(now, kind="stable"):
            if step(int(r)):
                break
        else:
            raise AssertionError("deadlock in the timing model")
    return float(now.max())
