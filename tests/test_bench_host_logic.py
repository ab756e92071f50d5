"""Host-side arithmetic of bench.py (no GPU): the algorithmic bytes behind the roofline figures and
the DRAM-traffic records that turn into roofline.traffic / roofline.dram_frac."""
import os

import numpy as np

import bench
import bls_inputs as bi

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_algorithmic_bytes_of_the_headline_workload():
    """26 tables x 1e6 rows x 64 fp32, batch 16384, about 20 IDs per bag: rows L * 256 B, IDs three times,
    bag boundaries three times, output once (fp32 [B][T][D])."""
    w = bi.workload(3)
    L = 8_519_243
    step, gather = bench.algorithmic_bytes(w, L)
    G = 16384 * 26
    assert step == L * 256 + 3 * L * 4 + 3 * G * 4 + G * 64 * 4
    assert gather == L * 256 + L * 4 + G * 4 + G * 64 * 4
    assert abs(step / 1e9 - 2.397) < 0.005 and abs(gather / 1e9 - 2.326) < 0.005
    # row-wise placement: every owner gets a boundary entry for every bag
    w4 = bi.workload(4)
    s4, g4 = bench.algorithmic_bytes(w4, 20_970_000)
    G4 = w4.n_bags
    assert g4 == 20_970_000 * 256 + 20_970_000 * 4 + G4 * w4.P * 4 + G4 * 128 * 4


def test_traffic_records_belong_to_the_committed_gather_source():
    """profiles/gather_traffic.json is only used while its hash matches the gather kernel's source:
    a change to that source without a new capture would silently blank roofline.traffic."""
    src = os.path.join(ROOT, "paper_2512_19342_b200", "csrc", "bls_gather.cu")
    for num, lo, hi in ((3, 0.5e9, 0.9e9), (4, 1.5e9, 2.6e9), (5, 1.8e9, 2.8e9)):
        t = bench.traffic_record(src, bi.workload(num).name)
        assert t is not None, f"no valid DRAM-traffic record for workload {num}: re-capture it"
        assert lo < t < hi
    assert bench.traffic_record(src, "no_such_workload") is None


def test_host_delay_draws_are_reproducible_and_uniform():
    d = bench.host_delay_draws(8, 4000, 600_000, 7)
    assert d.shape == (8, 4000) and d.min() >= 0 and d.max() <= 600_000
    assert np.array_equal(d, bench.host_delay_draws(8, 4000, 600_000, 7))
    assert abs(d.mean() - 300_000) < 5_000                      # uniform on [0, span]
    assert not np.array_equal(d[0], d[1])                       # ranks draw different sequences
