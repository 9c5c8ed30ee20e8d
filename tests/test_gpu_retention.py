"""Parity of the retention / refresh / wear part (hbf_enable_retention and friends) with the oracle's, through the C
ABI: integers bit for bit (plan order, claims, completions, counters), damage within 1e-12 relative (the two sides
call different exp() implementations)."""
import json
import os

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import hbfo
from paper_2609_09800_b200 import workloads as wl

BASE = wl.RANGE_BASE
PAGE = 16 * wl.KIB
RET = dict(pages_per_block=4, blocks_per_plane=8, blocks_per_zone=2, max_pec=3, disturb_limit=0,
           l_ref_s=1000.0, t_ref_c=40.0, ea_ev=1.04, accel=1.0, lead_threshold=0.5)


@pytest.fixture(scope="module")
def hbf():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_09800_b200 import build, hbf as mod
    build.build()
    return mod


def contexts(hbf, ret, geometry="tiny", floorplan=None, path=None, **over):
    prof = wl.load_profile("nominal", **wl.GEOMETRY[geometry])
    prof.update(over)
    g, o = hbf.Context(prof, floorplan), hbfo.Oracle(prof, floorplan)
    g.register_range(BASE, 64 * wl.GIB); o.register_range(BASE, 64 * wl.GIB)
    if path is not None:
        g.set_path(path)
    g.enable_retention(**ret); o.enable_retention(**ret)
    return g, o, prof


def compare_state(g, o, rtol=1e-12):
    bg, bo = g.retention_blocks(), o.retention_blocks()
    for k in ("disturb", "pec", "epoch"):
        bad = np.flatnonzero(bg[k] != bo[k])
        assert bad.size == 0, "%s: first mismatch at block %d: gpu %d oracle %d" % (k, bad[0], bg[k][bad[0]], bo[k][bad[0]])
    assert np.allclose(bg["damage"], bo["damage"], rtol=rtol, atol=0.0)
    assert g.retention_totals() == o.retention_totals()
    pg, po = g.retention_plan(), o.retention_plan()
    assert pg.shape == po.shape
    bad = np.flatnonzero(pg != po)
    assert bad.size == 0, "plan: first mismatch at %d: gpu %d oracle %d (%d of %d)" % (bad[0], pg[bad[0]], po[bad[0]], bad.size, pg.size)


def compare_batch(g, o, acc, rtol=1e-12):
    rc_o, c_o, s_o, st_o, ds_o = o.submit(acc, check=False)
    rc_g, c_g, s_g, st_g, ds_g = g.submit_host(acc, check=False)
    assert rc_g == rc_o
    if rc_o == 0:
        assert np.array_equal(st_g, st_o)
        bad = np.flatnonzero(c_g != c_o)
        assert bad.size == 0, "first mismatch at %d: gpu %d oracle %d (%d mismatches)" % (bad[0], c_g[bad[0]], c_o[bad[0]], bad.size)
        assert np.array_equal(s_g, s_o)
        for k in hbfo.DIE_STATS_DTYPE.names:
            assert np.array_equal(ds_g[k], ds_o[k]), k
        assert g.last_result() == o.last_result()
    assert np.array_equal(g.get_busy_until(), o.busy_until())
    assert np.array_equal(g.get_pending_energy(), o.pending_energy())
    compare_state(g, o, rtol)
    return rc_g


def recs(rows):
    a = np.zeros(len(rows), hbfo.ACCESS_DTYPE)
    for i, (off, issue, nbytes, op) in enumerate(rows):
        a[i] = (BASE + off, issue, nbytes, op)
    return a


def offset_of(prof, ret, ch, di, pl, block, page=0):
    C, D, P = prof["channels"], prof["dies"], prof["planes"]
    return (((((block * ret["pages_per_block"] + page) * P + pl) * D + di) * C + ch)) * PAGE


def test_hand_example(hbf, golden_dir):
    with open(os.path.join(golden_dir, "retention_examples.json")) as f:
        ex = json.load(f)
    ret = dict(RET, **ex["retention"])
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"]); prof.update(ex["geometry"])
    g = hbf.Context(prof)
    g.register_range(BASE, wl.GIB)
    g.enable_retention(**ret)
    g.submit_host(recs([(offset_of(prof, ret, b["channel"], b["die"], b["plane"], b["block"]), 0, 64, 0) for b in ex["eligible_blocks"]]))
    g.retention_advance(0, np.array([40.0]))
    assert g.retention_plan().tolist() == ex["plan"]
    rows = [(offset_of(prof, ret, 1, 1, pl, 0), 0, PAGE, 0) for pl in (0, 1)] + [(offset_of(prof, ret, 1, 0, 1, 0), 0, PAGE, 0)]
    _, comp, _, _, _ = g.submit_host(recs(rows))
    assert comp.tolist() == ex["claims"]["completion_first"]
    _, comp, _, _, _ = g.submit_host(recs([(offset_of(prof, ret, 1, 1, pl, 0), 1_000_000, PAGE, 0) for pl in (0, 1)]))
    assert comp.tolist() == ex["claims"]["completion_second"]
    pec = g.retention_blocks()["pec"]
    assert {str(i): int(v) for i, v in enumerate(pec) if v} == ex["claims"]["pec_after_second"]
    assert g.retention_plan().tolist() == ex["claims"]["plan_after_second"]
    g.retention_decay(ex["decay"]["idle_ns"])
    pec = g.retention_blocks()["pec"]
    assert {str(i): int(v) for i, v in enumerate(pec) if v} == ex["decay"]["pec_after"]
    assert g.retention_plan().tolist() == ex["decay"]["plan_after"]
    t = g.retention_totals()
    assert (t["planned"], t["claimed"], t["decayed"], t["commits"]) == (10, 5, 2, 3)


def mixed_batch(rng, n, t0, span_pages, natives=0.1, progs=0.1, gap=400):
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = BASE + rng.integers(0, span_pages, n).astype(np.uint64) * np.uint64(PAGE) + rng.integers(0, 4, n).astype(np.uint64) * np.uint64(4096)
    acc["issue_ns"] = t0 + np.sort(rng.integers(0, gap * n + 1, n))
    acc["bytes"] = rng.choice([64, 4096, 16000, 40000], n)
    acc["flags"] = rng.random(n) < progs
    nat = rng.random(n) < natives
    acc["addr"][nat] = 0x2000 + 64 * np.arange(int(nat.sum()), dtype=np.uint64)
    return acc


@pytest.mark.parametrize("path", ["auto", "sort"])
@pytest.mark.parametrize("n", [1, 33, 2049, 70_000])
def test_rounds_of_batches_epochs_and_decay(hbf, n, path):
    """Blocks become eligible by read disturb and by damage, batches claim what they can, blocks commit and wear out."""
    ret = dict(RET, disturb_limit=max(2, n // 300), lead_threshold=0.02, max_pec=2, pages_per_block=4)
    g, o, prof = contexts(hbf, ret, path=hbf.PATH_AUTO if path == "auto" else hbf.PATH_SORT)
    rng = np.random.default_rng(n + (7 if path == "sort" else 0))
    span_pages = 8 * 4 * 2 * 8 * 4 * 2                                   # twice the tracked blocks: the block index wraps
    t0 = 0
    for round_ in range(6):
        acc = mixed_batch(rng, n, t0, span_pages)
        assert compare_batch(g, o, acc) == 0
        t0 = int(acc["issue_ns"][-1]) + 50_000_000
        temps = np.array([rng.uniform(35.0, 95.0)])
        dt = int(rng.integers(1, 40)) * 10**9
        g.retention_advance(dt, temps); o.retention_advance(dt, temps)
        compare_state(g, o)
        if round_ % 2 == 1:
            idle = int(rng.integers(0, 30)) * 395_000 + int(rng.integers(0, 395_000))
            g.retention_decay(idle); o.retention_decay(idle)
            compare_state(g, o)
    t = o.retention_totals()
    if n >= 2049:                                                        # the scenario does exercise every stage
        assert t["claimed"] > 0 and t["commits"] > 0 and t["worn_blocks"] > 0


def test_whole_batch_claims_and_debt_remains(hbf):
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9, pages_per_block=64, blocks_per_plane=64, blocks_per_zone=8)
    g, o, prof = contexts(hbf, ret)
    rows = [(offset_of(prof, ret, c, d, 0, 0), 0, 64, 0) for c in range(8) for d in range(4)]
    compare_batch(g, o, recs(rows))
    g.retention_advance(0, np.array([40.0])); o.retention_advance(0, np.array([40.0]))
    compare_state(g, o)
    assert o.retention_totals()["planned"] == 32 * 64
    w = wl.tiny_uniform(n=1500, seed=4, rho=0.9)
    acc = w.acc.copy(); acc["issue_ns"] += 10**8
    assert compare_batch(g, o, acc) == 0
    assert o.retention_totals()["claimed"] == 1500
    acc["issue_ns"] += 10**9
    assert compare_batch(g, o, acc) == 0                                  # the debt ends inside this one
    assert o.retention_totals()["claimed"] == 2048


def test_thermally_scaled_claims(hbf):
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9)
    g, o, prof = contexts(hbf, ret)
    rng = np.random.default_rng(5)
    compare_batch(g, o, mixed_batch(rng, 500, 0, 4096, natives=0.0, progs=0.0))
    g.retention_advance(0, np.array([40.0])); o.retention_advance(0, np.array([40.0]))
    g.force_mode(1, 612_345); hbfo.lib().hbfo_force_mode(o._h, 1, 612_345)
    assert compare_batch(g, o, mixed_batch(rng, 3000, 10**9, 4096)) == 0
    idle = 10 * 395_000
    g.retention_decay(idle); o.retention_decay(idle)                      # the drain rate is scaled too
    compare_state(g, o)


def test_capacity_geometry_two_million_accesses(hbf):
    """2,048 queues, a batch of many tiles, the claim limit deep inside it, natives mixed in."""
    ret = dict(RET, pages_per_block=8, blocks_per_plane=16, blocks_per_zone=4, disturb_limit=3, lead_threshold=1e9, max_pec=100)
    g, o, prof = contexts(hbf, ret, geometry="capacity")
    rng = np.random.default_rng(9)
    n = 2_000_000
    span_pages = 64 * 8 * 4 * 16 * 8
    acc = mixed_batch(rng, n, 0, span_pages, gap=12)
    assert compare_batch(g, o, acc) == 0
    g.retention_advance(10**9, np.full(1, 50.0)); o.retention_advance(10**9, np.full(1, 50.0))
    compare_state(g, o)
    debt = o.retention_totals()["planned"]
    assert 50_000 < debt < n
    acc["issue_ns"] += 10**9
    assert compare_batch(g, o, acc) == 0
    assert o.retention_totals()["claimed"] == debt
    acc["issue_ns"] += 10**9
    assert compare_batch(g, o, acc) == 0                                  # no debt: the in-order path serves it


def test_region_temperatures_from_the_thermal_field(hbf):
    fp = wl.toy_floorplan(16, 48, 8, 4)
    ret = dict(RET, lead_threshold=1e9)
    g, o, prof = contexts(hbf, ret, floorplan=fp)
    rng = np.random.default_rng(2)
    ext = np.asarray(fp["ext_power_w"], np.float32) if "ext_power_w" in fp else None
    t0 = 0
    for _ in range(5):
        acc = mixed_batch(rng, 20_000, t0, 4096, gap=100)
        compare_batch(g, o, acc, rtol=2e-4)                              # 1e-3 K of field tolerance is 1.3e-4 of lifetime
        t0 = int(acc["issue_ns"][-1]) + 1
        g.thermal_step(1_000_000, ext); o.thermal_step(1_000_000, ext)
        g.retention_advance(10**9); o.retention_advance(10**9)
    bg, bo = g.retention_blocks(), o.retention_blocks()
    assert bo["damage"].max() > bo["damage"].min() > 0                    # regions differ in temperature
    assert np.allclose(bg["damage"], bo["damage"], rtol=2e-4)
    assert g.retention_totals() == o.retention_totals()


@pytest.mark.parametrize("rho_gap", [400, 40])
def test_forced_inorder_path_applies_the_claims(hbf, rho_gap):
    """The in-order kernels (serve, fix-up, straggle, re-serve) with claims; the dense case backlogs every queue."""
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9, pages_per_block=128)
    g, o, prof = contexts(hbf, ret, path=hbf.PATH_INORDER)
    rng = np.random.default_rng(3)
    acc = mixed_batch(rng, 50_000, 0, 65536, gap=rho_gap)               # touches every tracked block
    assert compare_batch(g, o, acc) == 0                                  # no debt yet
    g.retention_advance(0, np.array([40.0])); o.retention_advance(0, np.array([40.0]))
    for k in range(3):                                                    # the debt ends inside the third batch
        acc = mixed_batch(rng, 30_000, 10**9 * (k + 1) if rho_gap == 400 else int(acc["issue_ns"][-1]) + 1, 4096, gap=rho_gap)
        assert compare_batch(g, o, acc) == 0
    assert o.retention_totals()["claimed"] == o.retention_totals()["planned"] > 30_000


def test_unsorted_batch_with_debt_goes_to_the_sort_path_and_counts_claims_once(hbf):
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9)
    g, o, prof = contexts(hbf, ret)
    rng = np.random.default_rng(13)
    compare_batch(g, o, mixed_batch(rng, 20_000, 0, 4096))
    g.retention_advance(0, np.array([40.0])); o.retention_advance(0, np.array([40.0]))
    acc = mixed_batch(rng, 20_000, 10**9, 4096)
    acc = acc[rng.permutation(acc.shape[0])]                              # out of issue order: the in-order attempt is abandoned
    assert compare_batch(g, o, acc) == 0


def test_refused_batch_changes_nothing(hbf):
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9)
    g, o, prof = contexts(hbf, ret)
    compare_batch(g, o, recs([(0, 0, 64, 0), (PAGE * 9, 5, 64, 0)]))
    g.retention_advance(0, np.array([40.0])); o.retention_advance(0, np.array([40.0]))
    bad = recs([(PAGE, 10**7, 64, 0), (64 * wl.GIB - 32, 10**7, 64, 0), (2 * PAGE, 10**7, 64, 0)])
    assert compare_batch(g, o, bad) == hbfo.E_ACCESS_FAULT
    assert compare_batch(g, o, recs([(PAGE, 2 * 10**7, 64, 0)])) == 0


@pytest.mark.parametrize("path", ["auto", "sort"])
def test_with_the_energy_bins(hbf, path):
    """Claimed quanta are ledger events of their own; the ledger, the pending totals after thermal-clock steps and
    everything else stay bit-exact."""
    fp = wl.toy_floorplan(16, 48, 8, 4)
    ret = dict(RET, disturb_limit=2, lead_threshold=1e9, pages_per_block=16)
    g, o, prof = contexts(hbf, ret, floorplan=fp, path=hbf.PATH_AUTO if path == "auto" else hbf.PATH_SORT)
    g.enable_energy_bins(200_000, 16); o.enable_energy_bins(200_000, 16)
    rng = np.random.default_rng(21)
    t0 = 0
    for round_ in range(5):
        acc = mixed_batch(rng, 6000, t0, 4096, gap=300)
        assert compare_batch(g, o, acc) == 0
        fg, bg = g.energy_bins(); fo, bo = o.energy_bins()
        assert fg == fo and np.array_equal(bg, bo)
        t0 = int(acc["issue_ns"][-1]) + 1
        g.thermal_step(200_000); o.thermal_step(200_000)
        assert np.array_equal(g.get_pending_energy(), o.pending_energy())
        temps = np.full(len(fp["region_kind"]), 50.0)
        g.retention_advance(10**9, temps); o.retention_advance(10**9, temps)
        compare_state(g, o)
    assert o.retention_totals()["claimed"] > 1000


@pytest.mark.parametrize("path", ["auto", "sort"])
def test_with_the_channel_bus(hbf, path):
    ret = dict(RET, disturb_limit=2, lead_threshold=1e9, pages_per_block=16)
    g, o, prof = contexts(hbf, ret, path=hbf.PATH_AUTO if path == "auto" else hbf.PATH_SORT)
    g.enable_channel_bus(); o.enable_channel_bus()
    rng = np.random.default_rng(31)
    t0 = 0
    for round_ in range(4):
        acc = mixed_batch(rng, 8000, t0, 4096, gap=300)
        assert compare_batch(g, o, acc) == 0
        assert np.array_equal(g.get_bus_busy_until(), o.bus_busy_until())
        t0 = int(acc["issue_ns"][-1]) + 1
        g.retention_advance(10**9, np.array([50.0])); o.retention_advance(10**9, np.array([50.0]))
        compare_state(g, o)
    assert o.retention_totals()["claimed"] > 1000


def test_with_the_paged_submit_every_part_claims_and_disturbs_on_its_own(hbf):
    """The oracle's hand-worked case: a 32 KiB read is two parts on two channels; with two quanta owed both claim."""
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9, pages_per_block=2)
    g, o, prof = contexts(hbf, ret)
    first = recs([(offset_of(prof, ret, 5, 0, 0, 0), 0, 64, 0)])
    g.submit_host(first); o.submit(first)
    g.retention_advance(0, np.array([40.0])); o.retention_advance(0, np.array([40.0]))
    row = recs([(offset_of(prof, ret, 0, 0, 0, 0), 10**6, 2 * PAGE, 0)])
    _, c_g, s_g, _, ds_g = g.submit_host(row, parts_capacity=4)
    _, c_o, s_o, _, ds_o = o.submit(row, paged=True)
    assert c_g.tolist() == [10**6 + 415_683] and np.array_equal(c_g, c_o) and np.array_equal(s_g, s_o)
    assert g.retention_totals()["claimed"] == 2
    for k in hbfo.DIE_STATS_DTYPE.names:
        assert np.array_equal(ds_g[k], ds_o[k]), k
    assert np.array_equal(g.get_busy_until(), o.busy_until())
    compare_state(g, o)


def test_reset_clears_the_block_state(hbf):
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9)
    g, o, prof = contexts(hbf, ret)
    rng = np.random.default_rng(8)
    compare_batch(g, o, mixed_batch(rng, 3000, 0, 4096))
    g.retention_advance(10**9, np.array([60.0])); o.retention_advance(10**9, np.array([60.0]))
    g.reset(); hbfo.lib().hbfo_reset(o._h)
    compare_state(g, o)
    assert g.retention_totals()["planned"] == 0
    assert compare_batch(g, o, mixed_batch(rng, 3000, 0, 4096)) == 0


@pytest.mark.parametrize("geom", [dict(channels=3, dies=5, planes=3), dict(channels=4, dies=2, planes=2, queue_level=1),
                                  dict(channels=8, dies=4, planes=2, stripe_bytes=64 * wl.KIB)])
def test_other_geometries_and_two_ranges(hbf, geom):
    """Channel, die and plane counts that are not powers of two (division instead of masks), one queue per die, several
    pages per stripe unit, two registered ranges with media offsets of their own."""
    ret = dict(RET, disturb_limit=3, lead_threshold=0.05, pages_per_block=3, blocks_per_plane=12, blocks_per_zone=4)
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"]); prof.update(geom)
    g, o = hbf.Context(prof), hbfo.Oracle(prof)
    for c in (g, o):
        c.register_range(BASE, wl.GIB, 3, 0, 0, 5 * PAGE)
        c.register_range(BASE + 4 * wl.GIB, wl.GIB, 1, 0, 0, 3 * wl.GIB + 7 * PAGE)
    g.enable_retention(**ret); o.enable_retention(**ret)
    rng = np.random.default_rng(geom["channels"])
    t0 = 0
    for round_ in range(5):
        acc = mixed_batch(rng, 20_000, t0, 3000)
        second = rng.random(acc.shape[0]) < 0.4
        acc["addr"][second] += np.uint64(4 * wl.GIB)
        acc["flags"][second] = 0                                          # the second range is read-only
        assert compare_batch(g, o, acc) == 0
        t0 = int(acc["issue_ns"][-1]) + 10**8
        temps = np.array([rng.uniform(40.0, 90.0)])
        g.retention_advance(10**10, temps); o.retention_advance(10**10, temps)
        compare_state(g, o)
    t = o.retention_totals()
    assert t["claimed"] > 0 and t["commits"] > 0


def test_state_blob_carries_bus_ledger_and_retention(hbf):
    """Checkpoint and resume in the middle of a run with everything switched on (channel bus, energy bins, retention with
    outstanding debt): a fresh context that takes the blob serves the rest of the run exactly as the original does, which
    in turn is checked against the oracle throughout; a blob from a context with other things switched on is refused."""
    rng = np.random.default_rng(21)

    def batch(n, t0):
        a = np.zeros(n, hbfo.ACCESS_DTYPE)
        a["addr"] = BASE + rng.integers(0, 1 << 24, n).astype(np.uint64)
        a["issue_ns"] = t0 + np.sort(rng.integers(0, 3_000_000, n))
        a["bytes"] = rng.choice([64, 4096, 16384, 40_000], n)
        a["flags"] = rng.random(n) < 0.05
        return a
    ret = dict(RET, disturb_limit=3)

    def fresh():
        g, o, prof = contexts(hbf, ret)
        g.enable_channel_bus(); o.enable_channel_bus()
        g.enable_energy_bins(500_000, 32); o.enable_energy_bins(500_000, 32)
        return g, o
    g, o = fresh()
    compare_batch(g, o, batch(4000, 0))
    g.retention_advance(10**9, np.array([70.0])); o.retention_advance(10**9, np.array([70.0]))
    compare_batch(g, o, batch(50, 3_000_000))                # claims part of the debt; the rest stays outstanding
    assert g.retention_totals()["planned"] > g.retention_totals()["claimed"] > 0
    blob = g.get_state()
    later = [batch(3000, 6_000_000), batch(3000, 9_000_000)]
    g2, _ = fresh()
    g2.set_state(blob)
    for acc in later:
        compare_batch(g, o, acc)
        rc2, c2, s2, st2, ds2 = g2.submit_host(acc, check=False)
        rc1 = g.last_result()["code"]
        assert rc2 == rc1 and g2.last_result() == g.last_result()
        assert np.array_equal(g2.get_busy_until(), g.get_busy_until()) and np.array_equal(g2.get_bus_busy_until(), g.get_bus_busy_until())
        (f1, b1), (f2, b2) = g.energy_bins(), g2.energy_bins()
        assert f1 == f2 and np.array_equal(b1, b2)
        assert g2.retention_totals() == g.retention_totals() and np.array_equal(g2.retention_plan(), g.retention_plan())
        r1, r2 = g.retention_blocks(), g2.retention_blocks()
        for k in r1:
            assert np.array_equal(r1[k], r2[k]), k
    plain, _, _ = contexts(hbf, ret)                          # retention only: the blob does not fit
    with pytest.raises(hbf.HbfError):
        plain.set_state(blob)
