"""Parity of the channel-bus stage (hbf_enable_channel_bus) with the oracle's, through the C ABI, bit for bit."""
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


def contexts(hbf, profile, ranges, path=None):
    g, o = hbf.Context(profile), hbfo.Oracle(profile)
    for r in ranges:
        g.register_range(*r)
        o.register_range(*r)
    if path is not None:
        g.set_path(path)
    g.enable_channel_bus(); o.enable_channel_bus()
    return g, o


def compare(g, o, acc):
    rc_o, c_o, s_o, st_o, ds_o = o.submit(acc, check=False)
    rc_g, c_g, s_g, st_g, ds_g = g.submit_host(acc, check=False)
    assert rc_g == rc_o
    if rc_o not in (0, hbfo.E_ACCESS_FAULT):
        return rc_g
    assert np.array_equal(st_g, st_o)
    bad = np.flatnonzero(c_g != c_o)
    assert bad.size == 0, "first mismatch at %d: gpu %d oracle %d (%d mismatches)" % (bad[0], c_g[bad[0]], c_o[bad[0]], bad.size)
    assert np.array_equal(s_g, s_o)
    for k in hbfo.DIE_STATS_DTYPE.names:
        assert np.array_equal(ds_g[k], ds_o[k]), k
    assert np.array_equal(g.get_busy_until(), o.busy_until())
    assert np.array_equal(g.get_bus_busy_until(), o.bus_busy_until())
    assert g.last_result() == o.last_result()
    return rc_g


def test_hand_examples(hbf, golden_dir):
    with open(os.path.join(golden_dir, "channel_bus_examples.json")) as f:
        examples = json.load(f)["examples"]
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    for ex in examples:
        g = hbf.Context(prof)
        g.register_range(wl.RANGE_BASE, wl.GIB)
        g.enable_channel_bus()
        for rows, want in zip(ex["batches"], ex["completion"]):
            acc = np.zeros(len(rows), hbfo.ACCESS_DTYPE)
            for i, (off, issue, nbytes, op) in enumerate(rows):
                acc[i] = (wl.RANGE_BASE + off, issue, nbytes, op)
            _, comp, _, _, _ = g.submit_host(acc)
            assert comp.tolist() == want, ex["name"]
        assert int(g.get_bus_busy_until()[0]) == ex["bus_busy_ch0"], ex["name"]


@pytest.mark.parametrize("path", ["auto", "sort"])
@pytest.mark.parametrize("n", [1, 33, 2049, 70_000])
def test_dense_mixed_stream_in_two_batches(hbf, n, path):
    rng = np.random.default_rng(n)
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = wl.RANGE_BASE + rng.integers(0, 1 << 24, n).astype(np.uint64)
    acc["issue_ns"] = np.sort(rng.integers(0, 600 * n, n))                 # dense: the buses do get busy
    acc["bytes"] = rng.choice([64, 4096, 16000, 60000], n)
    acc["flags"] = rng.random(n) < 0.05
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    g, o = contexts(hbf, prof, [(wl.RANGE_BASE, wl.GIB, 3, 0, 0, 0)], hbf.PATH_AUTO if path == "auto" else hbf.PATH_SORT)
    cut = n // 2
    compare(g, o, acc[:cut])
    compare(g, o, acc[cut:])
    if n > 1000:
        plain = hbfo.Oracle(prof); plain.register_range(wl.RANGE_BASE, wl.GIB)
        assert (g.submit_host(acc[:cut])[1] > plain.submit(acc[:cut])[1]).sum() > 0    # the stage did make reads wait


def test_capacity_geometry_statuses_refusal_and_reset(hbf):
    w = wl.capacity_mode(n=300_000, seed=3, rho=0.9)
    g, o = contexts(hbf, w.profile, w.ranges)
    compare(g, o, w.acc[:200_000])
    compare(g, o, w.acc[200_000:])
    wf, wm = wl.mixed_status(9000, seed=6, faults=True), wl.mixed_status(9000, seed=6)
    g, o = contexts(hbf, wm.profile, wm.ranges)
    assert compare(g, o, wf.acc) == hbfo.E_ACCESS_FAULT and not g.get_bus_busy_until().any()
    compare(g, o, wm.acc)                                                   # natives, two ranges, gaps
    g.reset(); o.reset()
    assert not g.get_bus_busy_until().any()
    compare(g, o, wm.acc)
    rc_o, c_o, s_o, _, _ = o.submit(wm.acc, check=False, paged=True)          # the page-granular submit queues parts on the buses
    rc_g, c_g, s_g, _, _ = g.submit_host(wm.acc, check=False, parts_capacity=100_000)
    assert rc_g == rc_o == 0 and np.array_equal(c_g, c_o) and np.array_equal(s_g, s_o)
    assert np.array_equal(g.get_bus_busy_until(), o.bus_busy_until())


def test_with_the_energy_ledger_on(hbf):
    w = wl.tiny_uniform(30_000, seed=2, rho=0.9)
    g, o = contexts(hbf, w.profile, w.ranges)
    g.enable_energy_bins(50_000, 700); o.enable_energy_bins(50_000, 700)
    compare(g, o, w.acc)
    (fg, bg), (fo, bo) = g.energy_bins(), o.energy_bins()
    assert fg == fo and np.array_equal(bg, bo)                             # the ledger's events are the array intervals, bus or not


@pytest.mark.parametrize("path", ["auto", "sort"])
def test_completion_past_the_key_width_is_refused_before_anything_is_committed(hbf, path):
    """With the bus stage on, array-done times are 47-bit sort keys in this library.  A batch issued just below 2^47 ns
    completes beyond it: the library refuses it (HBF_E_INVAL) with outputs zeroed and queue, bus and energy state
    unchanged, and goes on serving; the oracle, which has no such bound, serves the batch."""
    w = wl.tiny_uniform(4000, seed=11)
    g, o = contexts(hbf, w.profile, w.ranges, hbf.PATH_AUTO if path == "auto" else hbf.PATH_SORT)
    compare(g, o, w.acc[:2000])
    late = w.acc[2000:].copy()
    late["issue_ns"] += (1 << 47) - 1 - int(late["issue_ns"].max())
    busy0, bus0, pend0 = g.get_busy_until(), g.get_bus_busy_until(), g.get_pending_energy()
    rc_g, c_g, s_g, _, ds_g = g.submit_host(late, check=False)
    assert rc_g == hbf.E_INVAL and not c_g.any() and not s_g.any() and not ds_g["n_read"].any()
    assert np.array_equal(g.get_busy_until(), busy0) and np.array_equal(g.get_bus_busy_until(), bus0)
    assert np.array_equal(g.get_pending_energy(), pend0)
    o_late = hbfo.Oracle(w.profile); o_late.register_range(*w.ranges[0]); o_late.enable_channel_bus()
    o_late.submit(w.acc[:2000])
    rc_o, c_o, *_ = o_late.submit(late, check=False)
    assert rc_o == 0 and int(c_o.max()) >= (1 << 47)
    compare(g, o, w.acc[2000:])                              # the refusal left the context usable and its state exact
