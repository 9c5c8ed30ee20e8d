"""Pins of the oracle's page-granular submit (every page of an access queued on its own).

Hand-worked examples, the reduction to the ordinary submit when no access crosses a page, conservation
laws, and an independent event-by-event simulation in plain Python on small random inputs."""
import json
import os

import numpy as np
import pytest

from oracle import hbfo
from paper_2609_09800_b200 import workloads as wl

BASE = wl.RANGE_BASE


def make(prof=None, ranges=None, **over):
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"]) if prof is None else dict(prof)
    prof.update(over)
    o = hbfo.Oracle(prof)
    for r in (ranges if ranges is not None else [(BASE, wl.GIB, 3, 0, 0, 0)]):
        o.register_range(*r)
    return o, prof


def recs(rows):
    a = np.zeros(len(rows), hbfo.ACCESS_DTYPE)
    for i, (off, issue, nbytes, op) in enumerate(rows):
        a[i] = (BASE + off, issue, nbytes, op)
    return a


def test_hand_examples(golden_dir):
    with open(os.path.join(golden_dir, "paged_examples.json")) as f:
        examples = json.load(f)["examples"]
    for ex in examples:
        o, _ = make(stripe_bytes=ex["stripe_bytes"])
        _, comp, stall, status, ds = o.submit(recs(ex["acc"]), paged=True)
        assert comp.tolist() == ex["completion"], ex["name"]
        assert stall.tolist() == ex["stall"], ex["name"]
        assert (status == hbfo.ST_READY).all()
        assert int(ds["busy_ns"].sum()) == ex["busy_ns"], ex["name"]
        for k in ("n_read", "n_prog", "bytes_read", "bytes_prog"):
            assert int(ds[k].sum()) == ex.get(k, 0), (ex["name"], k)
        r = o.last_result()
        assert r["n_modeled"] == len(ex["acc"]) and r["modeled_ns"] == sum(ex["stall"])
        assert r["max_completion_ns"] == max(ex["completion"]) and r["service_ns"] == ex["busy_ns"]


def test_equals_the_ordinary_submit_when_no_access_crosses_a_page():
    w = wl.tiny_uniform(20_000, seed=3)                     # 4 KiB reads on 4 KiB-aligned slots of 16 KiB pages
    a, b = make(w.profile, w.ranges)[0], make(w.profile, w.ranges)[0]
    for part in (w.acc[:9000], w.acc[9000:]):
        ra, rb = a.submit(part), b.submit(part, paged=True)
        for x, y in zip(ra[1:4], rb[1:4]):
            assert np.array_equal(x, y)
        for k in hbfo.DIE_STATS_DTYPE.names:
            assert np.array_equal(ra[4][k], rb[4][k]), k
        assert np.array_equal(a.busy_until(), b.busy_until())
        assert np.array_equal(a.pending_energy(), b.pending_energy())
        assert a.last_result() == b.last_result()


def simulate(prof, acc, busy0=None):
    """Event by event, in plain Python: parts are generated access by access and appended to per-queue lists that
    are already in (issue, index, part) order because the input is sorted by issue time."""
    C, D, P = prof["channels"], prof["dies"], prof["planes"]
    pg, stripe = prof["page_bytes"], prof["stripe_bytes"]
    busy = dict() if busy0 is None else dict(busy0)
    comp = []
    for addr, issue, nbytes, flags in acc.tolist():
        off, end, op = addr - BASE, addr - BASE + nbytes, flags & 1
        worst = None
        lo = off
        while lo < end:
            hi = min(end, (lo // pg + 1) * pg)
            u = lo // stripe
            qu = ((u % C) * D + (u // C) % D) * P + (u // (C * D)) % P
            gran = prof["prog_granule"] if op else prof["read_granule"]
            cb = -(-(hi - lo) // gran) * gran
            xfer = -(-cb * 1000 // prof["chan_bytes_per_us"])
            s = prof["t_prog_ns"] if op else prof["t_read_ns"]
            arrive = issue + xfer if op else issue
            start = max(arrive, busy.get(qu, 0))
            busy[qu] = start + s
            done = busy[qu] + (0 if op else xfer)
            worst = done if worst is None else max(worst, done)
            lo = hi
        comp.append(worst)
    return np.array(comp, np.int64), busy


@pytest.mark.parametrize("stripe", [16384, 65536])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_against_a_plain_python_simulation(stripe, seed):
    rng = np.random.default_rng(seed)
    n = 3000
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = BASE + rng.integers(0, 1 << 24, n).astype(np.uint64)
    acc["issue_ns"] = np.sort(rng.integers(0, 30_000_000, n))
    acc["bytes"] = rng.choice([1, 64, 100, 4096, 16384, 20000, 65536, 200_000], n)
    acc["flags"] = rng.random(n) < 0.1
    o, prof = make(stripe_bytes=stripe)
    busy = None
    for part in (acc[:1700], acc[1700:]):                  # the second batch starts on the queues the first one left
        _, comp, stall, _, ds = o.submit(part, paged=True)
        want, busy = simulate(prof, part, busy)
        assert np.array_equal(comp, want)
        assert np.array_equal(stall, want - part["issue_ns"])
    got = o.busy_until()
    assert all(int(got[q]) == b for q, b in busy.items())


def test_conservation_laws():
    w = wl.capacity_mode(n=50_000, seed=2)                  # reads of 128 B .. 64 KiB, 16 KiB pages, 64 KiB stripes
    o, prof = make(w.profile, w.ranges)
    _, comp, stall, status, ds = o.submit(w.acc, paged=True)
    off = w.acc["addr"] - np.uint64(BASE)
    pages = (off % np.uint64(16384) + w.acc["bytes"] + np.uint64(16383)) // np.uint64(16384)
    assert int(ds["n_read"].sum()) == int(pages.sum())              # one page operation per page touched
    assert int(ds["busy_ns"].sum()) == int(pages.sum()) * prof["t_read_ns"]
    assert int(ds["energy_pj"].sum()) == int(ds["n_read"].sum()) * prof["e_cmd_read_pj"] + int(ds["bytes_read"].sum()) * prof["e_byte_read_pj"]
    assert (comp >= w.acc["issue_ns"] + prof["t_read_ns"]).all()    # at least one page of array time
    # splitting never makes an access on otherwise idle queues slower than the whole-access model
    o2, _ = make(w.profile, w.ranges)
    one = w.acc[:1]
    assert o2.submit(one, paged=True)[1][0] <= make(w.profile, w.ranges)[0].submit(one)[1][0]


def test_refusal_and_natives():
    w = wl.mixed_status(4000, seed=9, faults=True)
    o, _ = make(w.profile, w.ranges)
    rc, comp, stall, status, ds = o.submit(w.acc, check=False, paged=True)
    assert rc == hbfo.E_ACCESS_FAULT and not comp.any() and not stall.any() and not o.busy_until().any()
    w = wl.mixed_status(4000, seed=9)
    rc, comp, stall, status, ds = o.submit(w.acc, paged=True)
    nat = status == hbfo.ST_NATIVE
    assert nat.any() and np.array_equal(comp[nat], w.acc["issue_ns"][nat]) and not stall[nat].any()
