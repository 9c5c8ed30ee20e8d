"""Parity of the page-granular submit (hbf_submit_batch_paged) with the oracle's, through the C ABI, bit for bit."""
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
    return g, o


def capacity_for(acc, page):
    return int((acc["bytes"].astype(np.int64) // page + 2).sum()) if acc.shape[0] else 0


def compare(g, o, acc, page=16384):
    rc_o, c_o, s_o, st_o, ds_o = o.submit(acc, check=False, paged=True)
    rc_g, c_g, s_g, st_g, ds_g = g.submit_host(acc, check=False, parts_capacity=capacity_for(acc, page))
    assert rc_g == rc_o
    if rc_o not in (0, hbfo.E_ACCESS_FAULT):               # refused for the mode: not classified, outputs not defined
        assert np.array_equal(g.get_busy_until(), o.busy_until())
        return rc_g
    assert np.array_equal(st_g, st_o)
    bad = np.flatnonzero(c_g != c_o)
    assert bad.size == 0, "first mismatch at %d: gpu %d oracle %d (%d mismatches)" % (bad[0], c_g[bad[0]], c_o[bad[0]], bad.size)
    assert np.array_equal(s_g, s_o)
    for k in hbfo.DIE_STATS_DTYPE.names:
        assert np.array_equal(ds_g[k], ds_o[k]), k
    assert np.array_equal(g.get_busy_until(), o.busy_until())
    assert np.array_equal(g.get_pending_energy(), o.pending_energy())
    assert g.last_result() == o.last_result()
    return rc_g


@pytest.mark.parametrize("path", ["auto", "sort"])
@pytest.mark.parametrize("n", [1, 2, 2047, 2048, 2049, 50_000, 300_001])
def test_capacity_mode_reads_of_one_to_five_pages(hbf, n, path):
    w = wl.capacity_mode(n=n, seed=n)
    g, o = contexts(hbf, w.profile, w.ranges, hbf.PATH_AUTO if path == "auto" else hbf.PATH_SORT)
    cut = n // 3
    compare(g, o, w.acc[:cut])
    compare(g, o, w.acc[cut:])


@pytest.mark.parametrize("stripe", [16384, 65536])
def test_mixed_sizes_programs_and_unaligned_spans(hbf, stripe):
    rng = np.random.default_rng(stripe)
    n = 40_000
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = wl.RANGE_BASE + rng.integers(0, 1 << 26, n).astype(np.uint64)
    acc["issue_ns"] = np.sort(rng.integers(0, 400_000_000, n))
    acc["bytes"] = rng.choice([1, 64, 100, 4096, 16384, 20000, 65536, 200_000, 1 << 20], n)
    acc["flags"] = rng.random(n) < 0.1
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"]); prof["stripe_bytes"] = stripe
    for path in (hbf.PATH_AUTO, hbf.PATH_SORT):
        g, o = contexts(hbf, prof, [(wl.RANGE_BASE, wl.GIB, 3, 0, 0, 0)], path)
        compare(g, o, acc[:25_000])
        compare(g, o, acc[25_000:])
    shuffled = acc[rng.permutation(n)]                       # any record order: the sort path
    g, o = contexts(hbf, prof, [(wl.RANGE_BASE, wl.GIB, 3, 0, 0, 0)])
    compare(g, o, shuffled)


def test_statuses_refusal_and_modes(hbf):
    wf, w = wl.mixed_status(9000, seed=6, faults=True), wl.mixed_status(9000, seed=6)
    g, o = contexts(hbf, w.profile, w.ranges)
    assert compare(g, o, wf.acc) == hbfo.E_ACCESS_FAULT    # refused: nothing changes
    compare(g, o, w.acc)                                     # natives, two ranges with gaps
    g.force_mode(hbf.MODE_LIGHT, 700_001); o.force_mode(hbfo.MODE_LIGHT, 700_001)
    compare(g, o, w.acc)
    g.force_mode(hbf.MODE_SEVERE, 700_001); o.force_mode(hbfo.MODE_SEVERE, 700_001)
    assert compare(g, o, w.acc) == hbfo.E_THROTTLED


def test_empty_batch_and_too_small_a_capacity(hbf):
    w = wl.capacity_mode(n=5000, seed=1)
    g, o = contexts(hbf, w.profile, w.ranges)
    compare(g, o, w.acc[:0])
    rc, *_ = g.submit_host(w.acc, check=False, parts_capacity=5000)     # these 5,000 reads have about 7,000 pages
    assert rc == hbf.E_WORKSPACE and not g.get_busy_until().any()
    compare(g, o, w.acc)


# ---- with the energy ledger, the channel bus and retention on: the list of parts is served like any batch of records ----

RET = dict(pages_per_block=4, blocks_per_plane=8, blocks_per_zone=2, max_pec=3, disturb_limit=40,
           l_ref_s=1000.0, t_ref_c=40.0, ea_ev=1.04, accel=1.0, lead_threshold=0.02)


def same_extras(g, o, bins, bus, ret):
    if bins:
        fg, bg = g.energy_bins(); fo, bo = o.energy_bins()
        assert fg == fo
        bad = np.argwhere(bg != bo)
        assert bad.size == 0, "bins: first difference at bin %d die %d: gpu %d oracle %d" % (bad[0][0], bad[0][1], bg[tuple(bad[0])], bo[tuple(bad[0])])
    if bus:
        assert np.array_equal(g.get_bus_busy_until(), o.bus_busy_until())
    if ret:
        bg, bo = g.retention_blocks(), o.retention_blocks()
        for k in ("disturb", "pec", "epoch"):
            assert np.array_equal(bg[k], bo[k]), k
        assert np.allclose(bg["damage"], bo["damage"], rtol=1e-12, atol=0.0)
        assert g.retention_totals() == o.retention_totals()
        assert np.array_equal(g.retention_plan(), o.retention_plan())


def busy_stream(rng, n, t0, gap):
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = wl.RANGE_BASE + rng.integers(0, 1 << 24, n).astype(np.uint64)
    acc["issue_ns"] = t0 + np.sort(rng.integers(0, gap * n + 1, n))
    acc["bytes"] = rng.choice([64, 4096, 16384, 20000, 65536, 200_000], n)
    acc["flags"] = rng.random(n) < 0.1
    nat = rng.random(n) < 0.05
    acc["addr"][nat] = 0x2000 + 64 * np.arange(int(nat.sum()), dtype=np.uint64)
    return acc


@pytest.mark.parametrize("path", ["auto", "sort"])
@pytest.mark.parametrize("extras", ["bins", "bus", "retention", "bins+bus+retention"])
def test_parts_with_the_ledger_the_bus_and_retention(hbf, extras, path):
    bins, bus, ret = "bins" in extras, "bus" in extras, "retention" in extras
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    g, o = contexts(hbf, prof, [(wl.RANGE_BASE, wl.GIB, 3, 0, 0, 0)], hbf.PATH_AUTO if path == "auto" else hbf.PATH_SORT)
    for x in (g, o):
        if bins:
            x.enable_energy_bins(250_000, 64)
        if bus:
            x.enable_channel_bus()
        if ret:
            x.enable_retention(**RET)
    rng = np.random.default_rng(len(extras))
    t0 = 0
    for n in (1, 4000, 30_000, 2049):
        acc = busy_stream(rng, n, t0, gap=4000)
        assert compare(g, o, acc) == 0
        same_extras(g, o, bins, bus, ret)
        t0 = int(acc["issue_ns"][-1]) + 1
        if ret:                                              # an epoch: disturbed blocks come due, the next batch's parts claim
            g.retention_advance(10**9, np.array([50.0])); o.retention_advance(10**9, np.array([50.0]))
            same_extras(g, o, bins, bus, ret)
    if ret:
        assert o.retention_totals()["claimed"] > 500
    if bus:
        assert o.bus_busy_until().any()
    if bins:
        assert o.energy_bins()[1].any()


def test_a_refused_paged_batch_changes_nothing_with_everything_on(hbf):
    wf = wl.mixed_status(6000, seed=4, faults=True)
    g, o = contexts(hbf, wf.profile, wf.ranges)
    for x in (g, o):
        x.enable_energy_bins(100_000, 64); x.enable_channel_bus(); x.enable_retention(**RET)
    assert compare(g, o, wf.acc) == hbfo.E_ACCESS_FAULT
    same_extras(g, o, True, True, True)
    assert not g.energy_bins()[1].any() and not g.get_bus_busy_until().any() and not g.retention_blocks()["disturb"].any()
