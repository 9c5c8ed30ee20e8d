"""Parity of the CUDA submit path with the CPU oracle, through the C ABI, element by element.

Integer outputs (completions, stalls, status, per-die stats, queue state, batch summary, served
order) must be bit-exact."""
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
    g = hbf.Context(profile)
    o = hbfo.Oracle(profile)
    for r in ranges:
        g.register_range(*r)
        o.register_range(*r)
    if path is not None:
        g.set_path(path)
    return g, o


def compare_batch(g, o, acc, check_order=False):
    rc_o, c_o, s_o, st_o, ds_o = o.submit(acc, check=False)
    rc_g, c_g, s_g, st_g, ds_g = g.submit_host(acc, check=False)
    assert rc_g == rc_o
    assert np.array_equal(st_g, st_o)
    bad = np.flatnonzero(c_g != c_o)
    assert bad.size == 0, "first mismatch at %d: gpu %d oracle %d (%d mismatches)" % (
        bad[0], c_g[bad[0]], c_o[bad[0]], bad.size)
    assert np.array_equal(s_g, s_o)
    for k in hbfo.DIE_STATS_DTYPE.names:
        assert np.array_equal(ds_g[k], ds_o[k]), k
    assert np.array_equal(g.get_busy_until(), o.busy_until())
    assert np.array_equal(g.get_pending_energy(), o.pending_energy())
    rg, ro = g.last_result(), o.last_result()
    assert rg == ro, (rg, ro)
    if check_order and rc_o == 0:
        assert np.array_equal(g.queue_order(acc.shape[0]), o.last_order())
    return rc_g


PATHS = ["auto", "sort", "sort_full"]


def path_id(hbf, name):
    return {"auto": hbf.PATH_AUTO, "sort": hbf.PATH_SORT, "sort_full": hbf.PATH_SORT_FULL}[name]


@pytest.mark.parametrize("path", PATHS)
def test_tiny_uniform_reads(hbf, path):
    w = wl.tiny_uniform()
    g, o = contexts(hbf, w.profile, w.ranges, path_id(hbf, path))
    compare_batch(g, o, w.acc, check_order=path != "auto")


@pytest.mark.parametrize("path", PATHS)
def test_mixed_status_shuffled(hbf, path):
    w = wl.mixed_status(10_000, seed=0)
    g, o = contexts(hbf, w.profile, w.ranges, path_id(hbf, path))
    compare_batch(g, o, w.acc[:6000], check_order=path != "auto")
    compare_batch(g, o, w.acc[6000:], check_order=path != "auto")          # queue state carries over


def test_faulting_batch_is_refused(hbf):
    w = wl.mixed_status(10_000, seed=0)
    wf = wl.mixed_status(10_000, seed=0, faults=True)
    g, o = contexts(hbf, w.profile, w.ranges)
    compare_batch(g, o, w.acc[:3000])
    assert compare_batch(g, o, wf.acc) == hbfo.E_ACCESS_FAULT
    compare_batch(g, o, w.acc[3000:])                    # the context stays usable, state untouched by the refusal


@pytest.mark.parametrize("n", [0, 1, 2, 31, 32, 33, 1023, 1024, 1025, 2047, 2048, 2049, 4095, 4096, 4097, 12289])
def test_ragged_sizes(hbf, n):
    w = wl.mixed_status(max(n, 1), seed=n)
    for path in (hbf.PATH_AUTO, hbf.PATH_SORT_FULL):
        g, o = contexts(hbf, w.profile, w.ranges, path)
        compare_batch(g, o, w.acc[:n], check_order=(path != hbf.PATH_AUTO and n > 0))


@pytest.mark.parametrize("path", PATHS)
def test_decode_weight_streaming(hbf, path):
    w = wl.decode_weights(tokens=4)
    g, o = contexts(hbf, w.profile, w.ranges, path_id(hbf, path))
    compare_batch(g, o, w.acc)


@pytest.mark.parametrize("path", PATHS)
def test_prefix_kv_programs_and_reads(hbf, path):
    w = wl.prefix_kv(epochs=2, steps=1, batch=16, kv_tokens=2048, layers=6)
    assert 0.005 < w.meta["frac_program"] < 0.2
    g, o = contexts(hbf, w.profile, w.ranges, path_id(hbf, path))
    cut = w.n // 3
    compare_batch(g, o, w.acc[:cut])
    compare_batch(g, o, w.acc[cut:])


@pytest.mark.parametrize("path", PATHS)
def test_capacity_mode_sizes(hbf, path):
    w = wl.capacity_mode(n=700_001)
    g, o = contexts(hbf, w.profile, w.ranges, path_id(hbf, path))
    compare_batch(g, o, w.acc)


def test_light_mode_scales_service(hbf):
    w = wl.prefix_kv(epochs=1, steps=1, batch=4, kv_tokens=1024, layers=3)
    g, o = contexts(hbf, w.profile, w.ranges)
    for q in (800_000, 999_999, 123_457, 1):
        g.force_mode(hbf.MODE_LIGHT, q); o.force_mode(hbfo.MODE_LIGHT, q)
        compare_batch(g, o, w.acc[:20_000])


def test_severe_and_shutdown_refuse(hbf):
    w = wl.tiny_uniform(3000)
    g, o = contexts(hbf, w.profile, w.ranges)
    compare_batch(g, o, w.acc[:1000])
    g.force_mode(hbf.MODE_SEVERE, 1_000_000); o.force_mode(hbfo.MODE_SEVERE, 1_000_000)
    rc_g = g.submit_host(w.acc[1000:2000], check=False)[0]
    rc_o = o.submit(w.acc[1000:2000], check=False)[0]
    assert rc_g == rc_o == hbfo.E_THROTTLED
    assert np.array_equal(g.get_busy_until(), o.busy_until())
    g.force_mode(hbf.MODE_NORMAL, 1_000_000); o.force_mode(hbfo.MODE_NORMAL, 1_000_000)
    compare_batch(g, o, w.acc[1000:2000])
    g.force_mode(hbf.MODE_SHUTDOWN, 1_000_000); o.force_mode(hbfo.MODE_SHUTDOWN, 1_000_000)
    assert g.submit_host(w.acc[2000:], check=False)[0] == o.submit(w.acc[2000:], check=False)[0] == hbfo.E_LINK_SHUTDOWN
    # terminal: the host side now refuses without launching
    assert g.submit_batch(None, 0, None, None) == hbf.E_LINK_SHUTDOWN


@pytest.mark.parametrize("geo", [dict(channels=3, dies=5, planes=2, page_bytes=4096, stripe_bytes=16384),
                                 dict(channels=8, dies=4, planes=2, page_bytes=16384, stripe_bytes=16384, queue_level=1),
                                 dict(channels=256, dies=16, planes=16, page_bytes=16384, stripe_bytes=16384),
                                 dict(channels=1, dies=1, planes=1, page_bytes=16384, stripe_bytes=16384)])
def test_other_geometries(hbf, geo):
    w = wl.mixed_status(30_000, seed=5)
    prof = dict(w.profile); prof.update(geo)
    for path in (hbf.PATH_AUTO, hbf.PATH_SORT_FULL):
        g, o = contexts(hbf, prof, w.ranges, path)
        compare_batch(g, o, w.acc, check_order=path != hbf.PATH_AUTO)


def test_equal_issue_times_and_hot_queue(hbf):
    # every access on one plane with many equal issue times: index order must decide
    rng = np.random.default_rng(3)
    n = 50_000
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = wl.RANGE_BASE + rng.integers(0, 4, n).astype(np.uint64) * np.uint64(4096)
    acc["issue_ns"] = rng.integers(0, 50, n)
    acc["bytes"] = rng.choice([64, 4096, 16384], n)
    acc["flags"] = rng.random(n) < 0.3
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    for path in (hbf.PATH_AUTO, hbf.PATH_SORT_FULL):
        g, o = contexts(hbf, prof, [(wl.RANGE_BASE, wl.GIB, 3, 0, 0, 0)], path)
        compare_batch(g, o, acc, check_order=path != hbf.PATH_AUTO)
        compare_batch(g, o, np.sort(acc, order="issue_ns", kind="stable"))


def test_large_issue_times_near_the_limit(hbf):
    w = wl.mixed_status(5000, seed=9)
    acc = w.acc.copy()
    acc["issue_ns"] += (1 << 47) - 1 - int(acc["issue_ns"].max())
    g, o = contexts(hbf, w.profile, w.ranges)
    compare_batch(g, o, acc)
    # one past the limit: the library's key width refuses the batch (its own restriction); the model has no such bound,
    # so the oracle serves the same batch
    late = np.sort(acc, order="issue_ns", kind="stable")
    late["issue_ns"][-1] = 1 << 47
    busy0, pend0 = g.get_busy_until(), g.get_pending_energy()
    rc_g, c_g, s_g, st_g, ds_g = g.submit_host(late, check=False)
    assert rc_g == hbf.E_ACCESS_FAULT and st_g[-1] == hbfo.ST_UNSUPPORTED and not c_g.any() and not s_g.any()
    assert np.array_equal(g.get_busy_until(), busy0) and np.array_equal(g.get_pending_energy(), pend0)
    rc_o, c_o, s_o, st_o, _ = o.submit(late, check=False)
    assert rc_o == 0 and st_o[-1] == st_o[-2] and c_o[-1] >= (1 << 47)
    g2, o2 = contexts(hbf, w.profile, w.ranges)
    compare_batch(g2, o2, acc)                              # a fresh pair still agrees below the limit


def test_argument_errors(hbf):
    import torch
    w = wl.tiny_uniform(100)
    g, _ = contexts(hbf, w.profile, w.ranges)
    d = torch.zeros(300, dtype=torch.int64, device="cuda")
    out = torch.zeros(100, dtype=torch.int64, device="cuda")
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    assert g.submit_batch(d, 100, out, out, d_workspace=small) == hbf.E_WORKSPACE
    assert g.submit_batch(None, 100, out, out) == hbf.E_INVAL
    assert g.submit_batch(d, 1 << 30, out, out) == hbf.E_INVAL
    assert g.register_range(wl.RANGE_BASE + 5, 10, check=False) == hbf.E_RANGE_OVERLAP
    assert g.workspace_bytes(1000) >= 1000 * 24


def test_state_blob_round_trip(hbf):
    w = wl.mixed_status(8000, seed=4)
    g, o = contexts(hbf, w.profile, w.ranges)
    compare_batch(g, o, w.acc[:4000])
    blob = g.get_state()
    g2, _ = contexts(hbf, w.profile, w.ranges)
    g2.set_state(blob)
    assert np.array_equal(g2.get_busy_until(), o.busy_until())
    compare_batch(g2, o, w.acc[4000:])
    with pytest.raises(hbf.HbfError):
        g2.set_state(blob[:-8])


# ---- the in-order path (batches whose records arrive in non-decreasing issue order) ---------------------

def issue_sorted(acc):
    return np.sort(acc, order="issue_ns", kind="stable")


@pytest.mark.parametrize("n", [1, 2, 2047, 2048, 2049, 4096, 10_000, 100_003])
def test_inorder_path_mixed_status(hbf, n):
    w = wl.mixed_status(n, seed=n + 1)
    acc = issue_sorted(w.acc)
    for path in (hbf.PATH_INORDER, hbf.PATH_AUTO, hbf.PATH_SORT):
        g, o = contexts(hbf, w.profile, w.ranges, path)
        cut = n // 2
        compare_batch(g, o, acc[:cut])
        compare_batch(g, o, acc[cut:])


def test_inorder_path_is_the_one_auto_takes(hbf):
    w = wl.tiny_uniform(30_000)
    g, o = contexts(hbf, w.profile, w.ranges, hbf.PATH_AUTO)
    compare_batch(g, o, w.acc)
    with pytest.raises(hbf.HbfError):                       # no sorted index array exists after an in-order batch
        g.queue_order(w.n)
    shuffled = w.acc[np.random.default_rng(0).permutation(w.n)]
    compare_batch(g, o, shuffled, check_order=True)         # falls back to the sort path


def test_forced_inorder_refuses_unsorted_batches(hbf):
    w = wl.mixed_status(5000, seed=3)
    g, o = contexts(hbf, w.profile, w.ranges, hbf.PATH_INORDER)
    rc, comp, stall, _, ds = g.submit_host(w.acc, check=False)
    assert rc == hbf.E_INVAL and not comp.any() and not stall.any() and not ds["busy_ns"].any()
    assert not g.get_busy_until().any()
    compare_batch(g, o, issue_sorted(w.acc))


def test_inorder_path_faults_and_throttle(hbf):
    wf = wl.mixed_status(9000, seed=6, faults=True)
    w = wl.mixed_status(9000, seed=6)
    g, o = contexts(hbf, w.profile, w.ranges, hbf.PATH_AUTO)
    assert compare_batch(g, o, issue_sorted(wf.acc)) == hbfo.E_ACCESS_FAULT
    g.force_mode(hbf.MODE_LIGHT, 700_001); o.force_mode(hbfo.MODE_LIGHT, 700_001)
    compare_batch(g, o, issue_sorted(w.acc))


def test_inorder_hot_queue_and_equal_issue(hbf):
    rng = np.random.default_rng(8)
    n = 60_000
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = wl.RANGE_BASE + rng.integers(0, 3, n).astype(np.uint64) * np.uint64(16384) + rng.integers(0, 4, n).astype(np.uint64) * np.uint64(4096)
    acc["issue_ns"] = np.sort(rng.integers(0, 2000, n))
    acc["bytes"] = rng.choice([64, 4096, 16384, 40000], n)
    acc["flags"] = rng.random(n) < 0.3
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    g, o = contexts(hbf, prof, [(wl.RANGE_BASE, wl.GIB, 3, 0, 0, 0)], hbf.PATH_INORDER)
    compare_batch(g, o, acc)
    compare_batch(g, o, acc)


def test_inorder_rows_with_lanes_on_one_queue(hbf):
    """The serve pass takes a row of 32 consecutive records at a time and has a path of its own for rows in which no two
    records share a queue, for rows with pairs only, and for rows where three or more do.  Every kind of row, built by
    hand on the 2,048 queues of the capacity geometry: no pair, one pair (neighbours, far apart, first and last lane),
    two and three pairs, a triple, four neighbours (the parts of a split access look like this), a triple beside a pair,
    all 32 on one queue, a pair broken by a record that is not modeled, and rows that repeat the queues of the row
    before."""
    rng = np.random.default_rng(21)
    labels = lambda pairs: [next((g for g, lanes in enumerate(pairs) if l in lanes), 100 + l) for l in range(32)]
    patterns = [labels([]), labels([(3, 4)]), labels([(2, 29)]), labels([(0, 31)]), labels([(1, 9), (10, 30)]),
                labels([(0, 1), (15, 16), (30, 31)]), labels([(5, 6, 20)]), labels([(8, 9, 10, 11)]),
                labels([(4, 12, 28), (7, 8)]), [0] * 32, labels([(13, 14)]), labels([(6, 7, 8, 9), (20, 21, 22, 23)])]
    rows, native_at = [], []
    prev_map = None
    for k in range(420):                                           # 13,440 records: beyond the small-batch route
        pat = patterns[int(rng.integers(0, len(patterns)))]
        if k % 7 == 3 and prev_map is not None:
            m = prev_map                                           # the same queues as in the row before
        else:
            units = rng.permutation(2048)
            m = {g: int(units[j]) for j, g in enumerate(sorted(set(range(200))))}
        prev_map = m
        rows.append([m[g] for g in pat])
        if pat == patterns[10]:
            native_at.append(32 * k + 13)                          # the first of the pair is outside every range
    unit = np.array(rows, np.uint64).reshape(-1)
    n = unit.shape[0]
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = np.uint64(wl.RANGE_BASE) + unit * np.uint64(65536) + rng.integers(0, 4, n).astype(np.uint64) * np.uint64(16384)
    acc["addr"][native_at] = 1 << 20
    acc["issue_ns"] = np.sort(rng.integers(0, 40_000_000, n))
    acc["issue_ns"][5000:5064] = acc["issue_ns"][5000]             # equal issue times across two rows
    acc["bytes"] = rng.choice([128, 4096, 16384], n)
    acc["flags"] = rng.random(n) < 0.2
    prof = wl.load_profile("nominal", **wl.GEOMETRY["capacity"])
    for path in (hbf.PATH_INORDER, hbf.PATH_SORT):
        g, o = contexts(hbf, prof, [(wl.RANGE_BASE, 2048 * 65536, 3, 0, 0, 0)], path)
        compare_batch(g, o, acc)
        compare_batch(g, o, acc)                                   # again, on the queues the first pass filled


@pytest.mark.parametrize("geo", [dict(channels=3, dies=5, planes=2, page_bytes=4096, stripe_bytes=16384),
                                 dict(channels=8, dies=4, planes=2, page_bytes=16384, stripe_bytes=16384, queue_level=1),
                                 dict(channels=32, dies=8, planes=8, page_bytes=16384, stripe_bytes=16384),
                                 dict(channels=1, dies=1, planes=1, page_bytes=16384, stripe_bytes=16384)])
def test_inorder_other_geometries(hbf, geo):
    w = wl.mixed_status(40_000, seed=5)
    prof = dict(w.profile); prof.update(geo)
    g, o = contexts(hbf, prof, w.ranges, hbf.PATH_INORDER)
    compare_batch(g, o, issue_sorted(w.acc))


def test_inorder_long_accesses(hbf):
    """Accesses with a service time beyond 32 bits of ns and a transfer of milliseconds, among ordinary ones; a service
    of 2^33 ns or more (a 512 MiB program: 12.3 s) sends the batch to the sort path, and is refused when the caller
    has declared the in-order path."""
    w = wl.tiny_uniform(20_000, seed=4)
    for nbytes, flags in ((32 << 20, 0), (256 << 20, 1), (512 << 20, 1)):
        acc = w.acc.copy()
        acc["bytes"][7777] = nbytes
        acc["flags"][7777] = flags
        acc["addr"][7777] = wl.RANGE_BASE                   # the whole span stays inside the 1 GiB range
        for path in (hbf.PATH_AUTO, hbf.PATH_INORDER, hbf.PATH_SORT):
            g, o = contexts(hbf, w.profile, w.ranges, path)
            if path == hbf.PATH_INORDER and nbytes == 512 << 20:
                rc, *_ = g.submit_host(acc, check=False)
                assert rc == hbf.E_INVAL and not g.get_busy_until().any()
                continue
            compare_batch(g, o, acc)
    g, o = contexts(hbf, w.profile, w.ranges, hbf.PATH_AUTO)
    g.force_mode(hbf.MODE_LIGHT, 3); o.force_mode(hbfo.MODE_LIGHT, 3)      # service scaled 333,334 times: 6.7 s per page read
    compare_batch(g, o, w.acc[:3000])


@pytest.mark.parametrize("rho", [0.8, 0.95, 1.2])
def test_inorder_long_busy_periods(hbf, rho):
    """Heavily loaded queues stay backlogged far past the first accesses of a tile: the straggle pass (a few
    such queues in a tile) and the re-serve pass (many of them) correct the as-if-idle results."""
    w = wl.tiny_uniform(400_000, seed=11, rho=rho)
    g, o = contexts(hbf, w.profile, w.ranges, hbf.PATH_INORDER)
    compare_batch(g, o, w.acc)
    w = wl.capacity_mode(n=1_500_000, seed=5, rho=rho)
    g, o = contexts(hbf, w.profile, w.ranges, hbf.PATH_INORDER)
    compare_batch(g, o, w.acc)


@pytest.mark.parametrize("entries", [1, 2, 3, 4, 5, 6])
def test_inorder_head_entries_do_not_change_results(hbf, entries):
    """How many of a (tile, queue)'s first accesses the streaming pass keeps for the correction pass is a matter of speed
    only (by default the library sets it from what earlier batches needed): with every fixed number the results are the
    oracle's, on lightly and on heavily loaded queues, twice in a row (the second batch finds every queue busy)."""
    for w in (wl.capacity_mode(n=600_000, seed=9, rho=0.5), wl.capacity_mode(n=600_000, seed=9, rho=0.85), wl.tiny_uniform(150_000, seed=2, rho=0.9)):
        g, o = contexts(hbf, w.profile, w.ranges, hbf.PATH_INORDER)
        g.set_head_entries(entries)
        compare_batch(g, o, w.acc)
        compare_batch(g, o, w.acc)
    g = hbf.Context(w.profile)
    with pytest.raises(hbf.HbfError):
        g.set_head_entries(7)


# ---- batches of at most 8,192 records in issue order take a route of their own (one launch, a block per 64 queues) ----

@pytest.mark.parametrize("n", [8191, 8192, 8193])
def test_small_batch_route_and_its_upper_end(hbf, n):
    """Both sides of the size at which the tiled kernels take over, each batch on the queues the one before left."""
    w = wl.mixed_status(3 * n, seed=n)
    acc = issue_sorted(w.acc)
    for path in (hbf.PATH_AUTO, hbf.PATH_INORDER):
        g, o = contexts(hbf, w.profile, w.ranges, path)
        for k in range(3):
            compare_batch(g, o, acc[k * n:(k + 1) * n])


@pytest.mark.parametrize("geo", [dict(channels=3, dies=5, planes=2, page_bytes=4096, stripe_bytes=16384),
                                 dict(channels=8, dies=4, planes=2, page_bytes=16384, stripe_bytes=16384, queue_level=1),
                                 dict(channels=64, dies=8, planes=4, page_bytes=16384, stripe_bytes=65536),
                                 dict(channels=1, dies=1, planes=1, page_bytes=16384, stripe_bytes=16384)])
def test_small_batches_other_geometries_and_thermal_scaling(hbf, geo):
    """30 queues (a slice that is not full), one queue per die, 2,048 queues (32 slices), a single queue; then the same
    with the service scaled (Eq. 3), which takes the general form of the terms."""
    w = wl.mixed_status(12_000, seed=11)
    prof = dict(w.profile); prof.update(geo)
    acc = issue_sorted(w.acc)
    g, o = contexts(hbf, prof, w.ranges, hbf.PATH_AUTO)
    compare_batch(g, o, acc[:5000])
    g.force_mode(hbf.MODE_LIGHT, 612_345); o.force_mode(hbfo.MODE_LIGHT, 612_345)
    compare_batch(g, o, acc[5000:])


def test_small_batch_all_on_one_queue_and_equal_issue_times(hbf):
    rng = np.random.default_rng(21)
    n = 8192
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = wl.RANGE_BASE + rng.integers(0, 4, n).astype(np.uint64) * np.uint64(4096)      # one page: one queue
    acc["issue_ns"] = np.sort(rng.integers(0, 50, n))
    acc["bytes"] = rng.choice([64, 4096, 9000], n)
    acc["flags"] = rng.random(n) < 0.3
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    g, o = contexts(hbf, prof, [(wl.RANGE_BASE, wl.GIB, 3, 0, 0, 0)], hbf.PATH_AUTO)
    compare_batch(g, o, acc)
    compare_batch(g, o, acc[:3000])                          # again, on the backlog


def test_small_batch_with_a_very_long_service(hbf):
    """A 512 MiB program (12.3 s of array time, beyond the 2^33 ns the tiled kernels' per-tile sums allow) among 3,000 ordinary
    reads: the small-batch route keeps services in 64 bits, so the batch is served even with the in-order path declared."""
    w = wl.tiny_uniform(3000, seed=14)
    acc = w.acc.copy()
    acc["bytes"][1234] = 512 << 20; acc["flags"][1234] = 1; acc["addr"][1234] = wl.RANGE_BASE
    for path in (hbf.PATH_AUTO, hbf.PATH_INORDER):
        g, o = contexts(hbf, w.profile, w.ranges, path)
        assert compare_batch(g, o, acc) == 0
        compare_batch(g, o, w.acc)                           # and the next batch behind it


def test_small_batch_out_of_order_faults_and_natives_only(hbf):
    w = wl.mixed_status(6000, seed=31)
    g, o = contexts(hbf, w.profile, w.ranges, hbf.PATH_AUTO)
    compare_batch(g, o, w.acc, check_order=True)             # shuffled: handed to the sort path from the device
    compare_batch(g, o, issue_sorted(w.acc))                 # and the small route again on what it left
    wf = wl.mixed_status(6000, seed=31, faults=True)
    assert compare_batch(g, o, issue_sorted(wf.acc)) == hbfo.E_ACCESS_FAULT
    nat = issue_sorted(w.acc).copy()
    nat["addr"] = 0x1000 + 64 * np.arange(nat.shape[0], dtype=np.uint64)        # nothing inside a range
    compare_batch(g, o, nat)
    g2, _ = contexts(hbf, w.profile, w.ranges, hbf.PATH_INORDER)
    rc, comp, stall, _, ds = g2.submit_host(w.acc, check=False)                  # declared in order, but it is not
    assert rc == hbf.E_INVAL and not comp.any() and not g2.get_busy_until().any()


def test_pinned_host_pipeline_equals_one_batch(hbf):
    """hbf_submit_host: copy-in, service and read-back of consecutive chunks on three streams of the library: for records
    in issue order the result (outputs, per-die totals, summary, queue state) is that of one batch; pageable buffers
    work too; a chunk with a fail-closed access is reported and leaves zeros."""
    import torch
    w = wl.capacity_mode(n=230_000, seed=4)
    g, o = contexts(hbf, w.profile, w.ranges)
    _, c_o, s_o, _, ds_o = o.submit(w.acc)
    n = w.n
    h_in = torch.from_numpy(w.acc.view(np.int64).reshape(-1)).pin_memory()
    h_c, h_s = torch.empty(n, dtype=torch.int64).pin_memory(), torch.empty(n, dtype=torch.int64).pin_memory()
    h_ds = torch.empty(g.n_dies * 6, dtype=torch.int64).pin_memory()
    for chunk in (50_000, 230_000, 7):
        if chunk == 7:
            n_use = 100                                      # many tiny chunks
        else:
            n_use = n
        g.reset()
        rc, summary = g.submit_pinned(h_in, n_use, h_c, h_s, h_ds, chunk=chunk)     # hbf_submit_host: returns when the results are home
        assert rc == 0 and summary["code"] == 0 and summary["n_modeled"] + summary["n_native"] == n_use
        if n_use == n:
            assert summary == o.last_result()
            assert np.array_equal(h_c.numpy(), c_o) and np.array_equal(h_s.numpy(), s_o)
            assert np.array_equal(h_ds.numpy().view(hbfo.DIE_STATS_DTYPE)["bytes_read"], ds_o["bytes_read"])
            assert np.array_equal(g.get_busy_until(), o.busy_until())
        else:
            o2 = hbfo.Oracle(w.profile)
            for r in w.ranges:
                o2.register_range(*r)
            _, c2, s2, _, _ = o2.submit(w.acc[:n_use])
            assert np.array_equal(h_c.numpy()[:n_use], c2) and np.array_equal(h_s.numpy()[:n_use], s2)
    # pageable buffers, and a refusal in the middle: the second chunk holds a zero-byte access
    bad = w.acc[:30_000].copy(); bad["bytes"][17_000] = 0
    h_bad = torch.from_numpy(bad.view(np.int64).reshape(-1))
    c2, s2 = torch.empty(30_000, dtype=torch.int64), torch.empty(30_000, dtype=torch.int64)
    g.reset()
    rc, summary = g.submit_pinned(h_bad, 30_000, c2, s2, None, chunk=10_000)
    assert rc == hbf.E_ACCESS_FAULT and summary["n_fault"] == 1
    assert not c2[10_000:20_000].any() and c2[:10_000].all() and c2[20_000:].all()
    o2 = hbfo.Oracle(w.profile); o2.register_range(*w.ranges[0])
    _, c_a, *_ = o2.submit(bad[:10_000]); _, c_b, *_ = o2.submit(bad[20_000:])
    assert np.array_equal(c2[:10_000].numpy(), c_a) and np.array_equal(c2[20_000:].numpy(), c_b)


@pytest.mark.parametrize("stage", [1, 2])
def test_bounded_waits_run_out_and_the_batch_is_given_up(hbf, stage):
    """The look-back waits of the sort path are bounded.  With a poll budget of a few hundred and one early tile silenced
    (test support of the library: nothing stalls for real), every tile behind it runs out of polls and returns: the batch's
    result is HBF_E_TIMEOUT, its outputs are zeroed, the queue state is untouched, the context is poisoned and refuses
    later batches, and hbf_reset brings it back."""
    w = wl.mixed_status(30_000, seed=12)                     # shuffled: several radix passes, 8 sort tiles, 15 scan tiles
    g, o = contexts(hbf, w.profile, w.ranges, hbf.PATH_SORT_FULL)
    compare_batch(g, o, w.acc[:5000])
    busy0, pend0 = g.get_busy_until(), g.get_pending_energy()
    g.debug_wait_test(poll_limit=300, stage=stage, tile=1)
    rc, c_g, s_g, _, ds_g = g.submit_host(w.acc[5000:], check=False)
    assert rc == hbf.E_TIMEOUT and not c_g.any() and not s_g.any() and not ds_g["n_read"].any()
    assert np.array_equal(g.get_busy_until(), busy0) and np.array_equal(g.get_pending_energy(), pend0)
    g.debug_wait_test()                                     # the switch is off again, but the context stays poisoned
    rc, *_ = g.submit_host(w.acc[5000:], check=False)
    assert rc == hbf.E_TIMEOUT
    assert np.array_equal(g.get_busy_until(), busy0)
    g.reset(); o.reset()
    compare_batch(g, o, w.acc)                              # usable again, and exact
