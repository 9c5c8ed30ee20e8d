"""Pins of the oracle's page-granular submit (every page of an access queued on its own).

Hand-worked examples, the reduction to the ordinary submit when no access crosses a page, conservation
laws, and an independent event-by-event simulation in plain Python on small random inputs; and the same with the
energy ledger, the channel bus and retention switched on, where every part is an event, a bus transfer, a claimant
and a disturbing read of its own (hand-worked, and the bus against a plain-Python queue)."""
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


# ---- with the energy ledger, the channel bus and retention on: parts are requests of their own there too --------

def test_with_the_energy_bins_every_part_is_an_event_on_its_own_die():
    """Example P1 again (four pages on channels 0..3, each served from 1,000 to 21,000 on die 0 of its channel) with bins
    of 10 us: every part's 16,384 x 84 = 1,376,256 pJ is split 9,000 : 10,000 : 1,000 over bins 0, 1, 2 of ITS die:
    floor(1,376,256 x 0.45) = 619,315, floor(1,376,256 x 0.5) = 688,128, the remainder 68,813.  One event for the whole
    access would put all 5.5 uJ on die 0, spread over 80 us."""
    o, prof = make(stripe_bytes=16384)
    o.enable_energy_bins(10_000, 16)
    o.submit(recs([(0, 1000, 65536, 0)]), paged=True)
    first, bins = o.energy_bins()
    assert first == 0
    for ch in range(4):
        assert bins[:4, ch * prof["dies"]].tolist() == [619_315, 688_128, 68_813, 0], ch
    assert int(bins.sum()) == 4 * 1_376_256
    assert not o.pending_energy().any()


def test_with_the_channel_bus_a_part_queues_on_the_bus_of_its_own_channel():
    """Access 0 reads 32 KiB from stripe unit 7: its parts lie on channel 7 and channel 0 (die 1).  Access 1 reads 16 KiB on
    channel 0, die 0.  All three arrays are done at 20,000.  Bus 0 takes the two transfers in the order of the list of
    parts (access 0 part 1, then access 1): 20,683 and 21,366; bus 7 is free: 20,683.  As one request access 0 would
    have queued 40,000 + 1,366 on channel 7 alone."""
    o, _ = make(stripe_bytes=16384)
    o.enable_channel_bus()
    _, comp, stall, _, _ = o.submit(recs([(7 * 16384, 0, 32768, 0), (0, 0, 16384, 0)]), paged=True)
    assert comp.tolist() == [20_683, 21_366] and stall.tolist() == [20_683, 21_366]
    bus = o.bus_busy_until()
    assert bus[0] == 21_366 and bus[7] == 20_683 and not bus[1:7].any()


def test_with_the_channel_bus_the_order_is_done_time_first():
    """Stripe of two pages: both parts of access 0 queue on one plane (done at 20,000 and 40,000); access 1 on another
    die of the same channel is done at 20,000 too.  Bus: part 0 (20,000 -> 20,683), access 1 (tie on the done time,
    later in the list: 20,683 -> 21,366), part 1 (40,000 -> 40,683)."""
    o, _ = make(stripe_bytes=32768)
    o.enable_channel_bus()
    _, comp, _, _, _ = o.submit(recs([(0, 0, 32768, 0), (8 * 32768, 0, 16384, 0)]), paged=True)
    assert comp.tolist() == [40_683, 21_366]
    assert o.bus_busy_until()[0] == 40_683


def simulate_with_bus(prof, acc, busy0, bus0):
    """The array stage part by part as in simulate(), then every channel's bus as a single server over its read parts in
    (array-done time, position in the list of parts) order."""
    C, D, P = prof["channels"], prof["dies"], prof["planes"]
    pg, stripe = prof["page_bytes"], prof["stripe_bytes"]
    busy, bus = dict(busy0), dict(bus0)
    comp = [None] * len(acc)
    waiting = {}
    slot = 0
    for i, (addr, issue, nbytes, flags) in enumerate(acc.tolist()):
        off, end, op = addr - BASE, addr - BASE + nbytes, flags & 1
        lo = off
        while lo < end:
            hi = min(end, (lo // pg + 1) * pg)
            u = lo // stripe
            ch = u % C
            qu = (ch * D + (u // C) % D) * P + (u // (C * D)) % P
            gran = prof["prog_granule"] if op else prof["read_granule"]
            cb = -(-(hi - lo) // gran) * gran
            xfer = -(-cb * 1000 // prof["chan_bytes_per_us"])
            s = prof["t_prog_ns"] if op else prof["t_read_ns"]
            start = max(issue + xfer if op else issue, busy.get(qu, 0))
            busy[qu] = start + s
            if op:
                comp[i] = busy[qu] if comp[i] is None else max(comp[i], busy[qu])
            else:
                waiting.setdefault(ch, []).append((busy[qu], slot, xfer, i))
            slot += 1
            lo = hi
    for ch, items in waiting.items():
        b = bus.get(ch, 0)
        for done, _, xfer, i in sorted(items):
            b = max(b, done) + xfer
            comp[i] = b if comp[i] is None else max(comp[i], b)
        bus[ch] = b
    return np.array(comp, np.int64), busy, bus


@pytest.mark.parametrize("stripe", [16384, 65536])
@pytest.mark.parametrize("seed", [0, 1])
def test_with_the_channel_bus_against_a_plain_python_queue(stripe, seed):
    rng = np.random.default_rng(100 + seed)
    n = 3000
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = BASE + rng.integers(0, 1 << 24, n).astype(np.uint64)
    acc["issue_ns"] = np.sort(rng.integers(0, 12_000_000, n))            # dense enough for the buses to queue
    acc["bytes"] = rng.choice([64, 4096, 16384, 20000, 65536, 200_000], n)
    acc["flags"] = rng.random(n) < 0.1
    o, prof = make(stripe_bytes=stripe)
    o.enable_channel_bus()
    busy, bus = {}, {}
    waited = 0
    for part in (acc[:1700], acc[1700:]):
        _, comp, stall, _, _ = o.submit(part, paged=True)
        want, busy, bus = simulate_with_bus(prof, part, busy, bus)
        assert np.array_equal(comp, want)
        assert np.array_equal(stall, want - part["issue_ns"])
        waited += int((want != simulate(prof, part, None)[0]).sum())
    assert waited > 100                                                    # the bus did hold transfers back
    got = o.bus_busy_until()
    assert all(int(got[ch]) == b for ch, b in bus.items())
