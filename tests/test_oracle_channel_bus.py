"""Pins of the oracle's channel-bus stage (a read's transfer queues on its channel's bus after the array time)."""
import json
import os

import numpy as np
import pytest

from oracle import hbfo
from paper_2609_09800_b200 import workloads as wl

BASE = wl.RANGE_BASE


def make(bus=True, **over):
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    prof.update(over)
    o = hbfo.Oracle(prof)
    o.register_range(BASE, wl.GIB)
    if bus:
        o.enable_channel_bus()
    return o, prof


def recs(rows):
    a = np.zeros(len(rows), hbfo.ACCESS_DTYPE)
    for i, (off, issue, nbytes, op) in enumerate(rows):
        a[i] = (BASE + off, issue, nbytes, op)
    return a


def test_hand_examples(golden_dir):
    with open(os.path.join(golden_dir, "channel_bus_examples.json")) as f:
        examples = json.load(f)["examples"]
    for ex in examples:
        o, _ = make()
        for rows, want in zip(ex["batches"], ex["completion"]):
            acc = recs(rows)
            _, comp, stall, _, _ = o.submit(acc)
            assert comp.tolist() == want, ex["name"]
            assert np.array_equal(stall, comp - acc["issue_ns"])
            r = o.last_result()
            assert r["max_completion_ns"] == max(want) and r["modeled_ns"] == int(stall.sum())
        assert int(o.bus_busy_until()[0]) == ex["bus_busy_ch0"], ex["name"]


def simulate_bus(prof, acc, comp_plain, bus0):
    """Plain Python: per channel, the reads in (array-done, index) order through one server."""
    C, stripe = prof["channels"], prof["stripe_bytes"]
    out = comp_plain.copy()
    bus = dict(bus0)
    rows = []
    for i, (addr, issue, nbytes, flags) in enumerate(acc.tolist()):
        if flags & 1:
            continue
        cb = -(-nbytes // prof["read_granule"]) * prof["read_granule"]
        xfer = -(-cb * 1000 // prof["chan_bytes_per_us"])
        rows.append((((addr - BASE) // stripe) % C, int(comp_plain[i]) - xfer, i, xfer))
    for ch, done, i, xfer in sorted(rows):
        start = max(done, bus.get(ch, 0))
        bus[ch] = start + xfer
        out[i] = bus[ch]
    return out, bus


@pytest.mark.parametrize("seed", [0, 1])
def test_against_a_plain_python_queue(seed):
    rng = np.random.default_rng(seed)
    n = 4000
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = BASE + rng.integers(0, 1 << 22, n).astype(np.uint64)
    acc["issue_ns"] = np.sort(rng.integers(0, 3_000_000, n))          # dense: the buses do get busy
    acc["bytes"] = rng.choice([64, 4096, 16000, 60000], n)
    acc["flags"] = rng.random(n) < 0.05
    plain, prof = make(bus=False)
    o, _ = make()
    bus = {}
    waited = 0
    for part in (acc[:2500], acc[2500:]):
        _, c_plain, _, _, ds_plain = plain.submit(part)                  # the array stage is the ordinary model's
        _, comp, stall, _, ds = o.submit(part)
        want, bus = simulate_bus(prof, part, c_plain, bus)
        assert np.array_equal(comp, want) and np.array_equal(stall, want - part["issue_ns"])
        assert (comp >= c_plain).all()
        waited += int((comp > c_plain).sum())
        for k in hbfo.DIE_STATS_DTYPE.names:
            assert np.array_equal(ds[k], ds_plain[k])                    # the array stage and its statistics are untouched
        assert np.array_equal(o.busy_until(), plain.busy_until())
    assert waited > 100
    got = o.bus_busy_until()
    assert all(int(got[ch]) == b for ch, b in bus.items())


def test_transfers_on_a_bus_never_overlap_and_sparse_reads_are_unchanged():
    w = wl.tiny_uniform(20_000, seed=8, rho=0.9)
    o, prof = make()
    _, comp, _, _, _ = o.submit(w.acc)
    xfer = -(-4096 * 1000 // prof["chan_bytes_per_us"])
    ch = ((w.acc["addr"] - np.uint64(BASE)) // np.uint64(prof["stripe_bytes"])) % np.uint64(prof["channels"])
    for c in range(prof["channels"]):
        ends = np.sort(comp[ch == c])
        assert (np.diff(ends) >= xfer).all()                             # each transfer holds the bus for its whole length
    sparse = w.acc[:2000].copy()
    sparse["issue_ns"] = np.arange(2000) * 100_000                       # one read every 100 us: nothing ever waits
    a, b = make()[0], make(bus=False)[0]
    assert np.array_equal(a.submit(sparse)[1], b.submit(sparse)[1])
    a.reset()
    assert not a.bus_busy_until().any()
