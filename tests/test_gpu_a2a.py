"""The stand-alone BLS alltoallv of bytes against the plain definition of an alltoallv
(numpy slicing), with up to k+1 requests in flight.  GPU only."""
import numpy as np
import pytest
import torch

import paper_2512_19342_b200 as bls

pytestmark = pytest.mark.gpu


def make_request(P, rng, max_seg, align=1):
    counts = (rng.integers(0, max_seg + 1, size=(P, P)) // align * align).astype(np.int64)
    counts[rng.random((P, P)) < 0.15] = 0                       # some empty segments
    gaps = rng.integers(0, 5, size=(P, P)).astype(np.int64) * align
    sd = np.cumsum(counts + gaps, axis=1) - counts               # segments in order, with holes between them
    stride = int((counts + gaps).sum(axis=1).max()) + 16
    send = rng.integers(0, 256, size=(P, stride), dtype=np.uint8)
    return send, counts, sd


def expected(send, counts, sd):
    """Definition of alltoallv: receiver dst gets the segments of src = 0..P-1 back to back."""
    P = counts.shape[0]
    return [np.concatenate([send[s, sd[s, d]:sd[s, d] + counts[s, d]] for s in range(P)]) for d in range(P)]


@pytest.mark.parametrize("P,k,max_seg,align", [(4, 0, 1000, 1), (8, 2, 70000, 1), (8, 4, 4096, 16), (1, 1, 33, 1), (32, 1, 300, 1)])
def test_alltoallv_matches_definition(P, k, max_seg, align):
    rng = np.random.Generator(np.random.PCG64(P * 100 + k))
    a2a = bls.A2a(P, k, P * max_seg + 64)
    pending = []
    for j in range(3 * (k + 1) + 1):
        if len(pending) == k + 1:                                # the ring is full: complete the oldest first
            want, jj = pending.pop(0)
            recv, rc, rd, req = a2a.wait()
            assert req == jj
            recv, rc, rd = recv.cpu().numpy(), rc.cpu().numpy(), rd.cpu().numpy()
            for d in range(P):
                assert np.array_equal(recv[d, :len(want[d])], want[d]), (jj, d)
        send, counts, sd = make_request(P, rng, max_seg, align)
        a2a.post(torch.from_numpy(send).cuda(), torch.from_numpy(counts).cuda(), torch.from_numpy(sd).cuda(),
                 int(counts.max()))
        pending.append((expected(send, counts, sd), j))
        last = (counts, sd)
    while pending:
        want, jj = pending.pop(0)
        recv, rc, rd, req = a2a.wait()
        assert req == jj
        recv = recv.cpu().numpy()
        for d in range(P):
            assert np.array_equal(recv[d, :len(want[d])], want[d])
    # receive-side counts and displacements of the last request
    counts, sd = last
    assert np.array_equal(rc.cpu().numpy(), counts.T)
    assert np.array_equal(rd.cpu().numpy(), np.cumsum(counts.T, axis=1) - counts.T)
    assert a2a.status() == bls.BLS_OK


def test_ring_and_capacity_limits():
    P, k = 2, 1
    a2a = bls.A2a(P, k, 256)
    send = torch.zeros(P, 512, dtype=torch.uint8, device="cuda")
    counts = torch.full((P, P), 64, dtype=torch.int64, device="cuda")
    sd = torch.tensor([[0, 64], [0, 64]], dtype=torch.int64, device="cuda")
    with pytest.raises(bls.BlsError):
        a2a.wait()                                               # nothing outstanding
    a2a.post(send, counts, sd, 64)
    a2a.post(send, counts, sd, 64)
    with pytest.raises(bls.BlsError) as e:
        a2a.post(send, counts, sd, 64)                           # k + 1 = 2 requests are already outstanding
    assert e.value.code == bls.BLS_ESTATE
    a2a.wait(); a2a.wait()
    assert a2a.status() == bls.BLS_OK
    big = torch.full((P, P), 200, dtype=torch.int64, device="cuda")      # 2 x 200 bytes > 256 per receiver
    sd2 = torch.tensor([[0, 200], [0, 200]], dtype=torch.int64, device="cuda")
    a2a.post(send, big, sd2, 200)
    a2a.wait()
    assert a2a.status() == bls.BLS_ENOSPC
    assert torch.ones(4, device="cuda").sum().item() == 4.0


def test_size_hint_below_the_largest_segment_does_not_truncate():
    """max_segment_bytes only sizes the launch: a segment longer than the hint is still copied whole."""
    P = 4
    rng = np.random.Generator(np.random.PCG64(77))
    send, counts, sd = make_request(P, rng, 300_000)
    a2a = bls.A2a(P, 0, int(counts.sum(axis=0).max()) + 64)
    a2a.post(torch.from_numpy(send).cuda(), torch.from_numpy(counts).cuda(), torch.from_numpy(sd).cuda(), 1000)
    recv, rc, rd, _ = a2a.wait()
    want = expected(send, counts, sd)
    recv = recv.cpu().numpy()
    for d in range(P):
        assert np.array_equal(recv[d, :len(want[d])], want[d])
    assert np.array_equal(rc.cpu().numpy(), counts.T)
    assert a2a.status() == bls.BLS_OK


def test_rejected_segment_counts_as_empty():
    """A segment that does not fit is reported, arrives nowhere, and the receive-side counts and
    displacements stay consistent with each other."""
    P = 2
    a2a = bls.A2a(P, 0, 256)
    send = torch.arange(512, dtype=torch.int32, device="cuda").to(torch.uint8).repeat(P, 1)
    counts = torch.tensor([[100, 10], [200, 10]], dtype=torch.int64, device="cuda")   # receiver 0: 100 fits, 200 more do not
    sd = torch.tensor([[0, 300], [0, 300]], dtype=torch.int64, device="cuda")
    a2a.post(send, counts, sd, 200)
    recv, rc, rd, _ = a2a.wait()
    assert a2a.status() == bls.BLS_ENOSPC                   # the rejected segment; the completion check also sees it missing
    assert rc.cpu().tolist() == [[100, 0], [10, 10]]
    assert rd.cpu().tolist() == [[0, 100], [0, 10]]
