"""Parity of the time-bin energy ledger (hbf_enable_energy_bins) with the oracle's: bins bit for bit, temperatures
within 1e-3 K when the thermal steps consume them."""
import json
import os

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import hbfo
from paper_2609_09800_b200 import workloads as wl


@pytest.fixture(scope="module")
def hbf():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_09800_b200 import build, hbf as mod
    build.build()
    return mod


def contexts(hbf, profile, ranges, fp=None, path=None):
    g, o = hbf.Context(profile, fp), hbfo.Oracle(profile, fp)
    for r in ranges:
        g.register_range(*r)
        o.register_range(*r)
    if path is not None:
        g.set_path(path)
    return g, o


def same_bins(g, o):
    fg, bg = g.energy_bins()
    fo, bo = o.energy_bins()
    assert fg == fo
    bad = np.argwhere(bg != bo)
    assert bad.size == 0, "first difference at bin %d die %d: gpu %d oracle %d" % (bad[0][0], bad[0][1], bg[tuple(bad[0])], bo[tuple(bad[0])])


def test_hand_examples(hbf, golden_dir):
    with open(os.path.join(golden_dir, "energy_bin_examples.json")) as f:
        examples = json.load(f)["examples"]
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    for ex in examples:
        g = hbf.Context(prof)
        g.register_range(wl.RANGE_BASE, wl.GIB)
        g.enable_energy_bins(ex["bin_ns"], len(ex["bins"]))
        acc = np.zeros(len(ex["acc"]), hbfo.ACCESS_DTYPE)
        for i, (off, issue, nbytes, op) in enumerate(ex["acc"]):
            acc[i] = (wl.RANGE_BASE + off, issue, nbytes, op)
        g.submit_host(acc)
        first, bins = g.energy_bins()
        assert first == 0 and bins[:, 0].tolist() == ex["bins"], ex["name"]
        assert not bins[:, 1:].any() and not g.get_pending_energy().any()


@pytest.mark.parametrize("path", ["auto", "sort"])
@pytest.mark.parametrize("bin_ns", [7_000, 1_000_000])
def test_mixed_stream_in_two_batches(hbf, bin_ns, path):
    rng = np.random.default_rng(bin_ns)
    n = 60_000
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = wl.RANGE_BASE + rng.integers(0, 1 << 26, n).astype(np.uint64)
    acc["issue_ns"] = np.sort(rng.integers(0, 40_000_000, n))
    acc["bytes"] = rng.choice([1, 64, 4096, 16384, 65536, 300_000], n)
    acc["flags"] = rng.random(n) < 0.05
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    g, o = contexts(hbf, prof, [(wl.RANGE_BASE, wl.GIB, 3, 0, 0, 0)], path=hbf.PATH_AUTO if path == "auto" else hbf.PATH_SORT)
    n_bins = 500                                              # the stream runs past the ring: its end collects the rest
    g.enable_energy_bins(bin_ns, n_bins); o.enable_energy_bins(bin_ns, n_bins)
    for part in (acc[:35_000], acc[35_000:]):
        rc_o, c_o, s_o, _, ds_o = o.submit(part)
        rc_g, c_g, s_g, _, ds_g = g.submit_host(part)
        assert np.array_equal(c_g, c_o) and np.array_equal(ds_g["energy_pj"], ds_o["energy_pj"])
        same_bins(g, o)
    _, bins = g.energy_bins()
    assert bins.sum() > 0 and not g.get_pending_energy().any()


def test_refused_batches_book_nothing(hbf):
    wf = wl.mixed_status(5000, seed=2, faults=True)
    g, o = contexts(hbf, wf.profile, wf.ranges)
    g.enable_energy_bins(100_000, 64); o.enable_energy_bins(100_000, 64)
    rc, *_ = g.submit_host(wf.acc, check=False)
    assert rc == hbf.E_ACCESS_FAULT and not g.energy_bins()[1].any()
    rc, *_ = g.submit_host(wf.acc, check=False, parts_capacity=100_000)     # the page-granular submit refuses it the same way
    assert rc == hbf.E_ACCESS_FAULT and not g.energy_bins()[1].any()


def test_thermal_steps_consume_the_bins(hbf):
    w = wl.prefix_kv(epochs=1, steps=1, batch=4, kv_tokens=256, layers=2)
    fp = wl.package_floorplan()
    g, o = contexts(hbf, w.profile, w.ranges, fp)
    g.enable_energy_bins(1_000_000, 16); o.enable_energy_bins(1_000_000, 16)
    ext = fp["ext_power_w"]
    k = 0
    for _, batch in wl.timed_batches(w, 12_000_000):
        g.submit_host(batch); o.submit(batch)
        same_bins(g, o)
        hot_g = g.thermal_step(1_000_000, ext)
        hot_o, _ = o.thermal_step(1_000_000, ext)
        assert np.abs(np.asarray(hot_g, np.float64) - hot_o).max() < 1e-3
        k += 1
    assert k >= 10
    same_bins(g, o)
    assert np.abs(g.get_temps().astype(np.float64) - o.temps()).max() < 1e-3
    with pytest.raises(hbf.HbfError):
        g.thermal_step(2_000_000, ext)                        # in binned mode a step is one bin long
    g.reset(); o.reset()
    same_bins(g, o)


@pytest.mark.parametrize("path", ["auto", "sort"])
def test_events_far_longer_than_the_ring(hbf, path):
    """A ring of two bins and events that span about five bins each (and, after a thermal step, events that begin before
    the ring): the bins the ring clamps into its first and last slot are booked in one step each on the device, and must
    add up to what the oracle's bin-by-bin walk gives."""
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    fp = wl.package_floorplan()
    g, o = contexts(hbf, prof, [(wl.RANGE_BASE, wl.GIB, 3, 0, 0, 0)], fp, path=hbf.PATH_AUTO if path == "auto" else hbf.PATH_SORT)
    bin_ns = 4_001                                            # a read of one page (20,000 ns) spans five or six bins
    g.enable_energy_bins(bin_ns, 2); o.enable_energy_bins(bin_ns, 2)
    rng = np.random.default_rng(5)
    n = 3000
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = wl.RANGE_BASE + rng.integers(0, 1 << 22, n).astype(np.uint64)
    acc["issue_ns"] = np.sort(rng.integers(0, 60_000, n))
    acc["bytes"] = rng.choice([64, 4096, 40_000], n)
    acc["flags"] = rng.random(n) < 0.1
    for part in (acc[:1500], acc[1500:]):
        o.submit(part); g.submit_host(part)
        same_bins(g, o)
        for _ in range(3):                                    # the clock moves on: later events begin before the ring
            g.thermal_step(bin_ns, fp["ext_power_w"]); o.thermal_step(bin_ns, fp["ext_power_w"])
        same_bins(g, o)
        assert np.array_equal(g.get_pending_energy(), o.pending_energy())


def test_refused_thermal_step_changes_nothing(hbf):
    """Bins on and a reduced-order model attached: a call the model must refuse (a field output is asked for) returns
    HBF_E_INVAL before anything is enqueued: the ledger rows, the clock's bin and the pending energy stay as they were."""
    w = wl.prefix_kv(epochs=1, steps=1, batch=4, kv_tokens=256, layers=2)
    fp = wl.package_floorplan()
    g, _ = contexts(hbf, w.profile, w.ranges, fp)
    g.enable_energy_bins(1_000_000, 8)
    g.submit_host(w.acc[:20_000])
    n_regions = len(fp["region_kind"])
    rom = hbf.Rom(np.zeros((2, 2)), np.zeros((2, n_regions)), np.zeros((3, 2)), stream=g.stream)
    g.attach_rom(rom, [hbf.KIND_HBF, hbf.KIND_HBM, hbf.KIND_GPU], 1_000_000)
    first0, bins0 = g.energy_bins()
    pend0 = g.get_pending_energy()
    assert bins0.any()
    import torch
    d_t = torch.zeros(fp["grid_h"] * fp["grid_w"], dtype=torch.float32, device="cuda")
    assert g.thermal_step(1_000_000, fp["ext_power_w"], d_temps_out=d_t, check=False) == hbf.E_INVAL
    assert g.thermal_step(2_000_000, fp["ext_power_w"], check=False) == hbf.E_INVAL
    first1, bins1 = g.energy_bins()
    assert first1 == first0 and np.array_equal(bins1, bins0) and np.array_equal(g.get_pending_energy(), pend0)
    g.thermal_step(1_000_000, fp["ext_power_w"])             # an accepted step consumes the clock's bin
    first2, bins2 = g.energy_bins()
    assert first2 == first0 + 1 and np.array_equal(bins2[:-1], bins0[1:])
