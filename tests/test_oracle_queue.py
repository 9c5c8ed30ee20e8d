"""Pins of the CPU oracle's access path (classification, decode, service terms, FIFO recurrence).

None of these re-types the oracle's formulas: they use hand-worked values, closed forms,
invariants, a separate event-driven simulator, exhaustive permutations and a queueing-theory mean.
"""
import itertools
import json
import os

import numpy as np
import pytest

from oracle import hbfo
from paper_2609_09800_b200 import workloads as wl

BASE = wl.RANGE_BASE


def make(profile=None, ranges=None, **over):
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"]) if profile is None else dict(profile)
    prof.update(over)
    o = hbfo.Oracle(prof)
    for r in (ranges if ranges is not None else [(BASE, wl.GIB, 3, 0, 0, 0)]):
        o.register_range(*r)
    return o


def recs(rows, base=BASE):
    a = np.zeros(len(rows), hbfo.ACCESS_DTYPE)
    for i, (off, issue, nbytes, op) in enumerate(rows):
        a[i] = (base + off, issue, nbytes, op)
    return a


# ---- hand examples and paper values -------------------------------------------------------------

def _examples(golden_dir):
    with open(os.path.join(golden_dir, "hand_examples.json")) as f:
        return json.load(f)["examples"]


def test_hand_examples(golden_dir):
    for ex in _examples(golden_dir):
        o = make(stripe_bytes=ex["stripe_bytes"])
        o.force_mode(hbfo.MODE_NORMAL if ex["q_ppm"] == 1000000 else hbfo.MODE_LIGHT, ex["q_ppm"])
        _, comp, stall, status, ds = o.submit(recs(ex["acc"]))
        assert comp.tolist() == ex["completion"], ex["name"]
        assert stall.tolist() == ex["stall"], ex["name"]
        assert (status == hbfo.ST_READY).all()
        assert int(ds["busy_ns"].sum()) == ex["busy_ns"], ex["name"]
        assert int(o.busy_until()[0]) == ex["busy_until"], ex["name"]
        assert int(o.busy_until()[1:].max()) == 0
        if "energy_pj" in ex:
            assert int(ds["energy_pj"].sum()) == ex["energy_pj"]
            assert int(o.pending_energy().sum()) == ex["energy_pj"]


def test_hand_examples_hold_at_any_time_origin(golden_dir):
    """The model knows no clock origin: the hand-worked examples moved to start far beyond 2^47 ns (no issue time is
    too late for the definition) give the same completions moved by the same amount, and the same stalls."""
    for shift in (1 << 47, (1 << 60) + 12345):
        for ex in _examples(golden_dir):
            o = make(stripe_bytes=ex["stripe_bytes"])
            o.force_mode(hbfo.MODE_NORMAL if ex["q_ppm"] == 1000000 else hbfo.MODE_LIGHT, ex["q_ppm"])
            acc = recs(ex["acc"])
            acc["issue_ns"] += shift
            _, comp, stall, status, ds = o.submit(acc)
            assert (status == hbfo.ST_READY).all()
            assert comp.tolist() == [c + shift for c in ex["completion"]], ex["name"]
            assert stall.tolist() == ex["stall"], ex["name"]
            assert int(ds["busy_ns"].sum()) == ex["busy_ns"] and int(o.busy_until()[0]) == ex["busy_until"] + shift


def test_thermal_service_scaling_eq3(golden_dir):
    with open(os.path.join(golden_dir, "paper_values.json")) as f:
        cases = json.load(f)["thermal_service_scaling"]["cases"]
    for s0, q, want in cases:
        o = make(t_read_ns=s0)
        assert o.service_terms(64, 1, 0, q)["s_ns"] == want


def test_closed_form_back_to_back_reads():
    # n reads issued together on one queue finish at k*tR + transfer, k = 1..n
    for n, nbytes in ((1, 64), (17, 4096), (300, 16384)):
        o = make()
        xfer = -(-nbytes * 1000 // 24000)
        _, comp, stall, _, ds = o.submit(recs([(0, 1000, nbytes, 0)] * n))
        assert comp.tolist() == [1000 + (k + 1) * 20000 + xfer for k in range(n)]
        assert int(ds["busy_ns"][0]) == n * 20000 and int(ds["n_read"][0]) == n


def test_decode_hand_example():
    o = make()
    d = o.decode(0x1234000, 4096)
    assert d == dict(channel=5, die=1, plane=0, row=18, page=18, npages=1, queue=42)


def test_decode_is_a_bijection_and_spreads_evenly():
    for geo in (dict(channels=8, dies=4, planes=2, page_bytes=16384, stripe_bytes=16384),
                dict(channels=3, dies=5, planes=2, page_bytes=4096, stripe_bytes=16384),
                dict(channels=32, dies=8, planes=4, page_bytes=16384, stripe_bytes=65536)):
        o = make(wl.load_profile("nominal", **geo))
        C_, D_, P_, S_ = geo["channels"], geo["dies"], geo["planes"], geo["stripe_bytes"]
        R = C_ * D_ * P_
        seen = set()
        for u in range(3 * R):
            d = o.decode(u * S_ + 5, 1)
            assert d["queue"] == (d["channel"] * D_ + d["die"]) * P_ + d["plane"]
            assert d["channel"] + C_ * (d["die"] + D_ * (d["plane"] + P_ * d["row"])) == u      # encode(decode(u)) = u
            assert d["page"] == d["row"] * (S_ // geo["page_bytes"])
            seen.add((d["queue"], d["row"]))
        assert len(seen) == 3 * R
        last = o.decode(S_ - 1, 1)
        assert last["queue"] == 0 and last["page"] == S_ // geo["page_bytes"] - 1
    # die-level queues
    o = make(queue_level=1)
    d = o.decode(0x1234000, 4096)
    assert d["queue"] == 5 * 4 + 1


def test_npages_counts_touched_pages():
    o = make()
    for off, nbytes in ((0, 1), (0, 16384), (0, 16385), (16383, 2), (100, 65536), (16384 * 3 + 1, 16384 * 2)):
        touched = (off + nbytes - 1) // 16384 - off // 16384 + 1
        assert o.decode(off, nbytes)["npages"] == touched


def test_granule_rounding_and_energy():
    o = make()
    t = o.service_terms(1, 1, 0)
    assert t["charged_bytes"] == 64 and t["energy_pj"] == 64 * 84 and t["xfer_ns"] == 3   # ceil(64000/24000)
    t = o.service_terms(65, 1, 0)
    assert t["charged_bytes"] == 128
    t = o.service_terms(1, 1, 1)
    assert t["charged_bytes"] == 4096 and t["energy_pj"] == 4096 * 840 and t["s_ns"] == 375000
    o = make(e_cmd_read_pj=1000)
    assert o.service_terms(64, 1, 0)["energy_pj"] == 1000 + 64 * 84


# ---- range classification (fail-closed boundary) -------------------------------------------------------

def test_classification_truth_table():
    L = 1 << 20
    o = make(ranges=[(BASE, L, 3, 0, 0, 0), (BASE + L, L, 1, 0, 0, L), (BASE + 4 * L, L, 2, 0, 0, 2 * L)])
    S = hbfo
    assert o.classify(BASE, 1)[0] == S.ST_READY
    assert o.classify(BASE - 1, 1)[0] == S.ST_NATIVE
    assert o.classify(BASE - 1, 2)[0] == S.ST_NATIVE            # classified by its effective address
    assert o.classify(BASE + L - 64, 64) == (S.ST_READY, 0)     # ends exactly at the range end
    assert o.classify(BASE + L - 64, 65)[0] == S.ST_FAULT_PARTIAL   # spills into the adjacent range
    assert o.classify(BASE + 2 * L - 1, 2)[0] == S.ST_FAULT_PARTIAL  # spills into a gap
    assert o.classify(BASE + 2 * L, 1)[0] == S.ST_NATIVE
    assert o.classify(BASE + L, 64, flags=1)[0] == S.ST_FAULT_PERM   # program to a read-only range
    assert o.classify(BASE + L, 64, flags=0) == (S.ST_READY, 1)
    assert o.classify(BASE + 4 * L, 64, flags=0)[0] == S.ST_FAULT_PERM  # read from a program-only range
    assert o.classify(BASE + 4 * L, 64, flags=1)[0] == S.ST_READY
    assert o.classify(BASE, 0)[0] == S.ST_UNSUPPORTED
    assert o.classify(BASE, 64, flags=2)[0] == S.ST_UNSUPPORTED
    assert o.classify(BASE, 64, issue_ns=-1)[0] == S.ST_UNSUPPORTED
    assert o.classify(BASE, 64, issue_ns=(1 << 47))[0] == S.ST_READY          # the definition has no upper bound
    assert o.classify(BASE, 64, issue_ns=(1 << 62))[0] == S.ST_READY
    # a range that ends at the top of the address space: a span that would wrap is a partial fault
    top = (1 << 64) - L
    o2 = make(ranges=[(top - L, L, 3, 0, 0, 0)])
    assert o2.register_range(top, L, check=False) == hbfo.E_INVAL      # base+length wraps to 0
    o3 = make(ranges=[(top - 1, L, 3, 0, 0, 0)])
    assert o3.classify(top - 1 + L - 8, 8)[0] == S.ST_READY
    assert o3.classify(top - 1 + L - 8, 9)[0] == S.ST_FAULT_PARTIAL
    assert o3.classify((1 << 64) - 1, 0xFFFFFFFF)[0] == S.ST_NATIVE


def test_register_range_errors():
    o = make(ranges=[(BASE, 4096, 3, 0, 0, 0)])
    assert o.register_range(BASE + 4095, 10, check=False) == hbfo.E_RANGE_OVERLAP
    assert o.register_range(BASE - 10, 11, check=False) == hbfo.E_RANGE_OVERLAP
    assert o.register_range(BASE + 4096, 10) == 1                     # adjacent is fine
    assert o.register_range(BASE + 8192, 0, check=False) == hbfo.E_INVAL
    assert o.register_range(BASE + 8192, 10, perms=0, check=False) == hbfo.E_INVAL
    o = make(ranges=[], capacity_bytes=1 << 20)
    assert o.register_range(BASE, 1 << 20, media_offset=1, check=False) == hbfo.E_CAPACITY
    assert o.register_range(BASE, 1 << 20) == 0
    o = make(ranges=[])
    for k in range(64):
        o.register_range(BASE + k * 4096, 4096)
    assert o.register_range(BASE + 64 * 4096, 4096, check=False) == hbfo.E_RANGE_FULL


def test_linear_scan_agrees_with_bisect_on_random_ranges():
    rng = np.random.default_rng(5)
    for _ in range(20):
        k = int(rng.integers(1, 30))
        cuts = np.sort(rng.choice(1 << 20, 2 * k, replace=False)).astype(np.uint64)
        rngs = [(BASE + int(cuts[2 * i]), int(cuts[2 * i + 1] - cuts[2 * i]), 3, 0, 0, 0) for i in range(k)]
        order = rng.permutation(k)
        o = make(ranges=[rngs[i] for i in order])
        starts = np.array([r[0] for r in rngs], dtype=np.uint64)
        for addr in rng.integers(BASE - 10, BASE + (1 << 20) + 10, 200):
            nbytes = int(rng.integers(1, 64))
            j = int(np.searchsorted(starts, np.uint64(addr), side="right")) - 1
            inside = j >= 0 and addr < rngs[j][0] + rngs[j][1]
            want = hbfo.ST_NATIVE if not inside else (
                hbfo.ST_READY if addr + nbytes <= rngs[j][0] + rngs[j][1] else hbfo.ST_FAULT_PARTIAL)
            assert o.classify(int(addr), nbytes)[0] == want


def test_fault_refuses_the_whole_batch_and_changes_nothing():
    w = wl.mixed_status(2000, seed=1, faults=False)
    wf = wl.mixed_status(2000, seed=1, faults=True)
    o = hbfo.Oracle(w.profile)
    for r in w.ranges:
        o.register_range(*r)
    o.submit(w.acc[:500])
    busy0, pend0 = o.busy_until(), o.pending_energy()
    rc, comp, stall, status, ds = o.submit(wf.acc, check=False)
    assert rc == hbfo.E_ACCESS_FAULT
    res = o.last_result()
    assert res["code"] == hbfo.E_ACCESS_FAULT and res["n_fault"] == 3 and res["n_modeled"] == 0
    assert not comp.any() and not stall.any() and not ds["busy_ns"].any()
    assert sorted(status[status > 1].tolist()) == [hbfo.ST_FAULT_PARTIAL, hbfo.ST_FAULT_PERM, hbfo.ST_UNSUPPORTED]
    assert (o.busy_until() == busy0).all() and (o.pending_energy() == pend0).all()


def test_native_rows_pass_through():
    w = wl.mixed_status(3000, seed=2)
    o = hbfo.Oracle(w.profile)
    for r in w.ranges:
        o.register_range(*r)
    _, comp, stall, status, ds = o.submit(w.acc)
    nat = status == hbfo.ST_NATIVE
    assert 200 < nat.sum() < 400
    assert (comp[nat] == w.acc["issue_ns"][nat]).all() and not stall[nat].any()
    res = o.last_result()
    assert res["n_native"] == nat.sum() and res["n_modeled"] == (~nat).sum()
    assert int(ds["n_read"].sum() + ds["n_prog"].sum()) == (~nat).sum()


def test_modes_refuse_batches():
    o = make()
    a = recs([(0, 0, 4096, 0)])
    o.force_mode(hbfo.MODE_SEVERE, 1000000)
    assert o.submit(a, check=False)[0] == hbfo.E_THROTTLED
    assert not o.busy_until().any()
    o.force_mode(hbfo.MODE_SHUTDOWN, 1000000)
    assert o.submit(a, check=False)[0] == hbfo.E_LINK_SHUTDOWN
    o.force_mode(hbfo.MODE_LIGHT, 800000)
    assert o.submit(a)[1][0] == 25171


# ---- invariants -----------------------------------------------------------------------------------------

def _check_invariants(o, acc, comp, stall, status, ds, busy_before):
    """completion >= arrival + service + post; service intervals on a queue are disjoint and follow
    (issue, index) order; busy time = sum of services; busy_until never decreases."""
    prof = o.cfg
    ready = np.flatnonzero(status == hbfo.ST_READY)
    per_queue = {}
    tot_s = 0
    for i in ready:
        rng_id = o.classify(int(acc["addr"][i]), int(acc["bytes"][i]), int(acc["flags"][i]), int(acc["issue_ns"][i]))[1]
        r = RANGES_OF[id(o)][rng_id]
        d = o.decode(r[5] + int(acc["addr"][i]) - r[0], int(acc["bytes"][i]))
        t = o.service_terms(int(acc["bytes"][i]), d["npages"], int(acc["flags"][i]) & 1, o.mode()[1])
        op = int(acc["flags"][i]) & 1
        post = 0 if op else t["xfer_ns"]
        arrive = int(acc["issue_ns"][i]) + (t["xfer_ns"] if op else 0)
        end = int(comp[i]) - post
        start = end - t["s_ns"]
        assert start >= arrive
        assert int(stall[i]) == int(comp[i]) - int(acc["issue_ns"][i])
        per_queue.setdefault(d["queue"], []).append((int(acc["issue_ns"][i]), int(i), start, end, arrive))
        tot_s += t["s_ns"]
    assert int(ds["busy_ns"].sum()) == tot_s
    busy_after = o.busy_until()
    assert (busy_after >= busy_before).all()
    for q, lst in per_queue.items():
        lst.sort()
        prev_end = int(busy_before[q])
        for issue, i, start, end, arrive in lst:
            assert start == max(arrive, prev_end)          # work conserving, never overlapping
            prev_end = end
        assert int(busy_after[q]) == prev_end
    untouched = np.setdiff1d(np.arange(busy_after.shape[0]), np.array(list(per_queue), dtype=np.int64))
    assert (busy_after[untouched] == busy_before[untouched]).all()


RANGES_OF = {}


def _oracle_for(w):
    o = hbfo.Oracle(w.profile)
    for r in w.ranges:
        o.register_range(*r)
    RANGES_OF[id(o)] = w.ranges
    return o


def test_invariants_on_mixed_stream():
    w = wl.mixed_status(1500, seed=3)
    o = _oracle_for(w)
    busy0 = o.busy_until()
    _, comp, stall, status, ds = o.submit(w.acc[:800])
    _check_invariants(o, w.acc[:800], comp, stall, status, ds, busy0)
    busy1 = o.busy_until()
    _, comp, stall, status, ds = o.submit(w.acc[800:])       # carries queue state across batches
    _check_invariants(o, w.acc[800:], comp, stall, status, ds, busy1)


def test_split_of_an_issue_sorted_stream_gives_identical_results():
    w = wl.tiny_uniform(6000, seed=4)
    o = _oracle_for(w)
    _, comp, stall, _, ds = o.submit(w.acc)
    for cut in (1, 2999, 5999):
        o2 = _oracle_for(w)
        _, c1, s1, _, d1 = o2.submit(w.acc[:cut])
        _, c2, s2, _, d2 = o2.submit(w.acc[cut:])
        assert (np.concatenate([c1, c2]) == comp).all() and (np.concatenate([s1, s2]) == stall).all()
        for k in hbfo.DIE_STATS_DTYPE.names:
            assert (d1[k] + d2[k] == ds[k]).all()
        assert (o2.busy_until() == o.busy_until()).all()


def test_later_batch_never_overtakes():
    o = make()
    o.submit(recs([(0, 100000, 4096, 0)]))
    _, comp, _, _, _ = o.submit(recs([(0, 0, 4096, 0)]))          # earlier issue time, later batch
    assert comp[0] == 120000 + 20000 + 171


# ---- an independent event-driven simulator, and exhaustive permutations ---------------------------------

def event_driven(queue_of, arrive, s, post, issue, busy0):
    """Advance time event by event; an idle server takes the head of its line (the line is kept in
    (issue, index) order) once that head has arrived.  Written independently of the oracle."""
    n = len(issue)
    lines = {}
    for i in sorted(range(n), key=lambda i: (issue[i], i)):
        lines.setdefault(queue_of[i], []).append(i)
    free_at = dict(busy0)
    done = [None] * n
    events = sorted(set(arrive) | set(free_at.values()) | {0})
    t_idx = 0
    now = events[0]
    pending = True
    while pending:
        pending = False
        nxt = None
        for q, line in lines.items():
            while line:
                head = line[0]
                fa = free_at.get(q, 0)
                if fa <= now and arrive[head] <= now:
                    free_at[q] = now + s[head]
                    done[head] = free_at[q] + post[head]
                    line.pop(0)
                    continue
                cand = max(fa, arrive[head])
                nxt = cand if nxt is None else min(nxt, cand)
                pending = True
                break
        if pending:
            now = nxt
    return done, free_at


def test_brute_force_tiny_batches():
    rng = np.random.default_rng(11)
    for trial in range(200):
        n = int(rng.integers(1, 9))
        rows = []
        for _ in range(n):
            q = int(rng.integers(0, 3))
            rows.append((q * 16384 + int(rng.integers(0, 8000)), int(rng.integers(0, 60000)),
                         int(rng.choice([64, 4096, 16384, 30000])), int(rng.random() < 0.3)))
        o = make()
        if trial % 3 == 0:
            o.submit(recs([(0, 0, 4096, 1)]))            # leaves queue 0 busy until 375171
        busy0 = {q: int(b) for q, b in enumerate(o.busy_until())}
        acc = recs(rows)
        _, comp, _, _, _ = o.submit(acc)
        qs, arr, ss, posts = [], [], [], []
        for off, issue, nbytes, op in rows:
            d = o.decode(off, nbytes)
            t = o.service_terms(nbytes, d["npages"], op)
            qs.append(d["queue"]); ss.append(t["s_ns"])
            arr.append(issue + (t["xfer_ns"] if op else 0)); posts.append(0 if op else t["xfer_ns"])
        done, free_at = event_driven(qs, arr, ss, posts, [r[1] for r in rows], busy0)
        assert comp.tolist() == done, (trial, rows)
        bu = o.busy_until()
        for q in set(qs):
            assert int(bu[q]) == free_at[q]


def test_all_permutations_of_a_distinct_issue_batch_agree():
    rows = [(0, 10, 4096, 0), (100, 5000, 20000, 1), (16384, 7, 64, 0), (0, 30000, 16384, 0),
            (200, 9000, 4096, 1), (16384, 90000, 4096, 0)]
    ref = None
    for perm in itertools.permutations(range(len(rows))):
        o = make()
        _, comp, stall, _, ds = o.submit(recs([rows[p] for p in perm]))
        by_row = {p: (int(comp[k]), int(stall[k])) for k, p in enumerate(perm)}
        sig = ([by_row[p] for p in range(len(rows))], o.busy_until().tolist(), ds["busy_ns"].tolist())
        if ref is None:
            ref = sig
        assert sig == ref


def test_queue_order_is_issue_then_index():
    w = wl.mixed_status(4000, seed=8)
    o = _oracle_for(w)
    _, _, _, status, _ = o.submit(w.acc)
    order = o.last_order()
    ready = np.flatnonzero(status == hbfo.ST_READY)
    assert np.array_equal(np.sort(order), ready)
    q = np.array([o.decode(RANGES_OF[id(o)][o.classify(int(a["addr"]), int(a["bytes"]), int(a["flags"]), int(a["issue_ns"]))[1]][5]
                           + int(a["addr"]) - RANGES_OF[id(o)][o.classify(int(a["addr"]), int(a["bytes"]), int(a["flags"]), int(a["issue_ns"]))[1]][0],
                           int(a["bytes"]))["queue"] for a in w.acc[order]])
    keys = list(zip(q.tolist(), w.acc["issue_ns"][order].tolist(), order.tolist()))
    assert keys == sorted(keys)


# ---- queueing theory: M/D/1 mean wait ----------------------------------------------------------------------

def test_md1_mean_wait_on_the_tiny_uniform_stream():
    # Poisson arrivals at load 0.5 on deterministic 20 us servers: mean wait = rho*s / (2(1-rho)) = 10 us
    w = wl.tiny_uniform(65536, seed=0)
    o = _oracle_for(w)
    _, comp, stall, status, ds = o.submit(w.acc)
    wait = stall - 20000 - 171
    assert (wait >= 0).all()
    assert abs(wait.mean() - 10000.0) / 10000.0 < 0.05
    per_queue = np.bincount([(a - BASE) // 16384 % 64 for a in w.acc["addr"].tolist()], minlength=64)
    assert abs(per_queue - 1024).max() < 5 * 32                  # uniform addresses load every plane alike


def test_config_validation():
    bad = [dict(channels=0), dict(page_bytes=3000), dict(stripe_bytes=8192), dict(queue_level=2),
           dict(t_read_ns=0), dict(chan_bytes_per_us=0), dict(q_light_ppm=0), dict(read_granule=48),
           dict(channels=1024, dies=1024)]
    for over in bad:
        with pytest.raises(hbfo.OracleError):
            make(**over)
