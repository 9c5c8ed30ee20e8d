"""Pins of the oracle's time-bin power integration (event energy split across bins by time overlap)."""
import json
import os

import numpy as np
import pytest

from oracle import hbfo
from paper_2609_09800_b200 import workloads as wl

BASE = wl.RANGE_BASE


def single_node_plan(n_dies, C=1000.0, Gs=1.0, idle=5.0):
    return dict(grid_h=1, grid_w=1, cell_C=[C], cell_Gx=[0.0], cell_Gy=[0.0], cell_Gsink=[Gs],
                cell_region=[0], die_region=[0] * n_dies, region_kind=[wl.KIND_HBF], region_idle_w=[idle])


def make(fp=None, **over):
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    prof.update(over)
    o = hbfo.Oracle(prof, fp)
    o.register_range(BASE, wl.GIB)
    return o, prof


def recs(rows):
    a = np.zeros(len(rows), hbfo.ACCESS_DTYPE)
    for i, (off, issue, nbytes, op) in enumerate(rows):
        a[i] = (BASE + off, issue, nbytes, op)
    return a


def test_hand_examples(golden_dir):
    with open(os.path.join(golden_dir, "energy_bin_examples.json")) as f:
        examples = json.load(f)["examples"]
    for ex in examples:
        o, _ = make()
        o.enable_energy_bins(ex["bin_ns"], len(ex["bins"]))
        _, _, _, _, ds = o.submit(recs(ex["acc"]))
        first, bins = o.energy_bins()
        assert first == 0
        assert bins[:, 0].tolist() == ex["bins"], ex["name"]
        assert not bins[:, 1:].any()
        assert int(ds["energy_pj"].sum()) == sum(ex["bins"])            # the per-die statistics are unchanged
        assert not o.pending_energy().any()                             # nothing is charged at submit any more


def test_every_die_keeps_its_energy_and_events_stay_inside_their_interval():
    w = wl.tiny_uniform(30_000, seed=5, rho=0.8)                        # 4 KiB reads, queues often busy
    o, prof = make()
    span = int(w.acc["issue_ns"].max()) + 10_000_000
    bin_ns = 50_000
    o.enable_energy_bins(bin_ns, span // bin_ns + 1)
    _, comp, _, _, ds = o.submit(w.acc)
    _, bins = o.energy_bins()
    assert np.array_equal(bins.sum(axis=0), ds["energy_pj"])
    # a read's event is the 20 us before its transfer: the energy booked up to any bin edge lies between the energy
    # of the events that ended before the edge and that of the events that started before it
    xfer = -(-4096 * 1000 // prof["chan_bytes_per_us"])
    end = comp - xfer
    start = end - prof["t_read_ns"]
    e = 84 * 4096
    cum = np.cumsum(bins.sum(axis=1))
    for k in (3, 40, 200, len(cum) - 2):
        edge = (k + 1) * bin_ns
        assert e * int((end <= edge).sum()) <= cum[k] <= e * int((start < edge).sum())


def test_time_outside_the_ring_is_booked_at_its_ends():
    o, _ = make()
    o.enable_energy_bins(10_000, 3)
    o.submit(recs([[0, 5000, 4096, 0]]))                                # [5000, 25000) fits bins 0..2
    o.submit(recs([[16384, 100_000, 4096, 0]]))                         # bins 10..11 -> the ring's last bin (other channel, die 4)
    _, bins = o.energy_bins()
    assert bins[:, 0].tolist() == [86016, 172032, 86016] and bins[:, 4].tolist() == [0, 0, 344064]
    o2, prof = make(single_node_plan(32), n_sub=1)
    o2.enable_energy_bins(10_000, 3)
    o2.thermal_step(10_000); o2.thermal_step(10_000)                     # the thermal clock now stands in bin 2
    o2.submit(recs([[0, 5000, 4096, 0]]))                                # bins 0..2: the past is booked into bin 2
    first, bins = o2.energy_bins()
    assert first == 2 and bins[:, 0].tolist() == [344064, 0, 0]


def test_a_step_consumes_the_bin_the_clock_stands_in():
    o, prof = make(single_node_plan(32, idle=5.0), n_sub=1)
    o.enable_energy_bins(1_000_000, 4)
    acc = recs([[0, 0, 16384, 0], [0, 1_200_000, 16384, 0]])            # one read per bin 0 and bin 1, 20 us each
    o.submit(acc)
    e = 84 * 16384
    rises = []
    for k in range(3):
        hot, _ = o.thermal_step(1_000_000)
        rises.append(hot[0])
    # one node, C = 1000 J/K, G_sink = 1 W/K, starting at ambient 35 C: T' = T + dt/C (P - G (T - 35)), P = E/dt + idle
    T, want = 35.0, []
    for E in (e, e, 0):
        P = E * 1e-12 / 1e-3 + 5.0
        T = T + 1e-3 / 1000.0 * (P - 1.0 * (T - 35.0))
        want.append(T)
    assert np.allclose(rises, want, rtol=0, atol=1e-12)
    first, bins = o.energy_bins()
    assert first == 3 and not bins.any()
    with pytest.raises(hbfo.OracleError):
        o.thermal_step(2_000_000)                                        # in binned mode a step is one bin long
    o.reset()
    assert o.energy_bins()[0] == 0
