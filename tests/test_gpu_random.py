"""Randomised parity: configurations drawn at random (geometry, granules, number of ranges, permissions, path, thermal
scaling, batch sizes with ragged tails, natives, faults; for retention also the block layout, thresholds, epochs and
idle-time decay in random order), every result compared with the oracle's, integers bit for bit."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import hbfo
from paper_2609_09800_b200 import workloads as wl

BASE = wl.RANGE_BASE


@pytest.fixture(scope="module")
def hbf():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_09800_b200 import build, hbf as mod
    build.build()
    return mod


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_configurations_and_batches(hbf, seed, cases=20):
    rng = np.random.default_rng(seed)
    bad = []
    for case in range(cases):
        pow2 = rng.random() < 0.7
        geo = dict(channels=int(rng.choice([1, 2, 8, 64] if pow2 else [3, 5, 12])), dies=int(rng.choice([1, 4, 8] if pow2 else [3, 6])),
                   planes=int(rng.choice([1, 2, 4] if pow2 else [3, 5])), page_bytes=int(rng.choice([4096, 16384])), queue_level=int(rng.random() < 0.2))
        geo["stripe_bytes"] = geo["page_bytes"] * int(rng.choice([1, 4]))
        prof = wl.load_profile("nominal", **geo)
        prof["read_granule"] = int(rng.choice([1, 64, 512])); prof["prog_granule"] = int(rng.choice([64, 4096]))
        nranges = int(rng.choice([1, 1, 1, 2, 3]))
        g, o = hbf.Context(prof), hbfo.Oracle(prof)
        span = 1 << 30
        for k in range(nranges):
            perms = int(rng.choice([3, 3, 1]))
            args = (BASE + k * 4 * span, span, perms, 0, 0, int(rng.integers(0, 1 << 20)) * 4096)
            g.register_range(*args); o.register_range(*args)
        path = [hbf.PATH_AUTO, hbf.PATH_AUTO, hbf.PATH_INORDER, hbf.PATH_SORT][int(rng.integers(0, 4))]
        g.set_path(path)
        if rng.random() < 0.3:
            q = int(rng.integers(200_000, 1_000_000)); g.force_mode(1, q); hbfo.lib().hbfo_force_mode(o._h, 1, q)
        t0 = 0
        for batch in range(int(rng.integers(1, 4))):
            n = int(rng.choice([1, 63, 64, 65, 1000, 50_001, 300_017, 1_200_003]))
            acc = np.zeros(n, hbfo.ACCESS_DTYPE)
            k = rng.integers(0, nranges, n).astype(np.uint64)
            acc["addr"] = BASE + k * np.uint64(4 * span) + rng.integers(0, span // 64, n).astype(np.uint64) * np.uint64(64)
            gap = float(rng.choice([5, 50, 500]))
            acc["issue_ns"] = t0 + np.sort(rng.integers(0, int(gap * n) + 1, n))
            acc["bytes"] = rng.choice([1, 64, 100, 4096, 16384, 65536, 200_000], n)
            acc["flags"] = rng.random(n) < float(rng.choice([0.0, 0.1, 0.5]))
            kind = rng.random()
            if kind < 0.25:
                nat = rng.random(n) < 0.2; acc["addr"][nat] = 4096 * np.arange(int(nat.sum()), dtype=np.uint64)
            faulty = rng.random() < 0.15
            if faulty:
                j = int(rng.integers(0, n)); what = int(rng.integers(0, 3))
                if what == 0: acc["bytes"][j] = 0
                elif what == 1: acc["flags"][j] = 2
                else: acc["addr"][j] = BASE + span - 8; acc["bytes"][j] = 64
            rc_o, c_o, s_o, st_o, ds_o = o.submit(acc, check=False)
            rc_g, c_g, s_g, st_g, ds_g = g.submit_host(acc, check=False)
            ok = rc_g == rc_o and np.array_equal(st_g, st_o) and np.array_equal(c_g, c_o) and np.array_equal(s_g, s_o) \
                and all(np.array_equal(ds_g[f], ds_o[f]) for f in hbfo.DIE_STATS_DTYPE.names) \
                and np.array_equal(g.get_busy_until(), o.busy_until()) and g.last_result() == o.last_result() \
                and np.array_equal(g.get_pending_energy(), o.pending_energy())
            if not ok:
                bad.append((case, batch, geo, nranges, path, n, rc_g, rc_o))
            t0 = int(acc["issue_ns"][-1]) + int(rng.integers(0, 10**6))
        g.destroy()
    assert not bad, bad


def retention_state_equal(g, o):
    bg, bo = g.retention_blocks(), o.retention_blocks()
    return all(np.array_equal(bg[k], bo[k]) for k in ("disturb", "pec", "epoch")) and np.allclose(bg["damage"], bo["damage"], rtol=1e-12, atol=0) \
        and g.retention_totals() == o.retention_totals() and np.array_equal(g.retention_plan(), o.retention_plan())


@pytest.mark.parametrize("seed", [21, 22, 23])
def test_random_retention_scenarios(hbf, seed, cases=20):
    rng = np.random.default_rng(seed)
    bad = []
    same = retention_state_equal
    for case in range(cases):
        pow2 = rng.random() < 0.7
        geo = dict(channels=int(rng.choice([2, 8, 16] if pow2 else [3, 5])), dies=int(rng.choice([1, 4] if pow2 else [3])),
                   planes=int(rng.choice([1, 2, 4] if pow2 else [3])), page_bytes=int(rng.choice([4096, 16384])), queue_level=int(rng.random() < 0.2))
        geo["stripe_bytes"] = geo["page_bytes"] * int(rng.choice([1, 4]))
        prof = wl.load_profile("nominal", **geo)
        bpz = int(rng.choice([1, 2, 4])); bpp = bpz * int(rng.choice([1, 3, 8]))
        ret = dict(pages_per_block=int(rng.choice([1, 3, 16])), blocks_per_plane=bpp, blocks_per_zone=bpz, max_pec=int(rng.choice([1, 2, 50])),
                   disturb_limit=int(rng.choice([0, 1, 5, 40])), l_ref_s=1000.0, t_ref_c=40.0, ea_ev=1.04, accel=float(rng.choice([1.0, 30.0])),
                   lead_threshold=float(rng.choice([0.05, 0.5, 1e9])))
        g, o = hbf.Context(prof), hbfo.Oracle(prof)
        g.register_range(BASE, 1 << 30); o.register_range(BASE, 1 << 30)
        g.set_path([hbf.PATH_AUTO, hbf.PATH_INORDER, hbf.PATH_SORT][int(rng.integers(0, 3))])
        g.enable_retention(**ret); o.enable_retention(**ret)
        if rng.random() < 0.3: g.enable_channel_bus(); o.enable_channel_bus()
        t0 = 0
        for step in range(int(rng.integers(3, 9))):
            what = rng.random()
            if what < 0.55:
                n = int(rng.choice([1, 64, 999, 20_001, 150_003]))
                acc = np.zeros(n, hbfo.ACCESS_DTYPE)
                acc["addr"] = BASE + rng.integers(0, 1 << 16, n).astype(np.uint64) * np.uint64(4096)
                acc["issue_ns"] = t0 + np.sort(rng.integers(0, 300 * n + 1, n))
                acc["bytes"] = rng.choice([64, 4096, 16384, 50_000], n)
                acc["flags"] = rng.random(n) < 0.15
                if rng.random() < 0.3:
                    nat = rng.random(n) < 0.2; acc["addr"][nat] = 4096 * np.arange(int(nat.sum()), dtype=np.uint64)
                if rng.random() < 0.1: acc["bytes"][int(rng.integers(0, n))] = 0
                if rng.random() < 0.3:
                    q = int(rng.integers(300_000, 1_000_001)); g.force_mode(1 if q < 1_000_000 else 0, q); hbfo.lib().hbfo_force_mode(o._h, 1 if q < 1_000_000 else 0, q)
                rc_o, c_o, s_o, st_o, ds_o = o.submit(acc, check=False)
                rc_g, c_g, s_g, st_g, ds_g = g.submit_host(acc, check=False)
                ok = rc_g == rc_o and (rc_o != 0 or (np.array_equal(c_g, c_o) and np.array_equal(s_g, s_o) and np.array_equal(st_g, st_o)
                     and all(np.array_equal(ds_g[f], ds_o[f]) for f in hbfo.DIE_STATS_DTYPE.names) and g.last_result() == o.last_result())) \
                     and np.array_equal(g.get_busy_until(), o.busy_until()) and np.array_equal(g.get_pending_energy(), o.pending_energy())
                t0 = int(acc["issue_ns"][-1]) + int(rng.integers(0, 10**7))
            elif what < 0.85:
                dt = int(rng.integers(0, 50)) * 10**9; temps = np.array([rng.uniform(30.0, 100.0)])
                g.retention_advance(dt, temps); o.retention_advance(dt, temps); ok = True
            else:
                idle = int(rng.integers(0, 5_000_000)); g.retention_decay(idle); o.retention_decay(idle); ok = True
            ok = ok and same(g, o)
            if not ok:
                bad.append((case, step, geo, ret)); break
        g.destroy()
    assert not bad, bad
