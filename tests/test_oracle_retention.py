"""Pins of the oracle's retention / refresh / wear part (Design D4): the Arrhenius lifetime and the damage sum
against closed forms, the plan order against a hand-worked example and against an independent formulation by
sorting, the debt claims against runs without debt, commits, wear-out and the fail-closed rule."""
import json
import os

import numpy as np
import pytest

from oracle import hbfo
from paper_2609_09800_b200 import workloads as wl

BASE = wl.RANGE_BASE
PAGE = 16 * wl.KIB
RET = dict(pages_per_block=4, blocks_per_plane=8, blocks_per_zone=2, max_pec=3, disturb_limit=0,
           l_ref_s=1000.0, t_ref_c=40.0, ea_ev=1.04, accel=1.0, lead_threshold=0.5)


def make(ret=None, floorplan=None, **over):
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    prof.update(over)
    o = hbfo.Oracle(prof, floorplan)
    o.register_range(BASE, wl.GIB)
    if ret is not None:
        o.enable_retention(**ret)
    return o, prof


def recs(rows):
    a = np.zeros(len(rows), hbfo.ACCESS_DTYPE)
    for i, (off, issue, nbytes, op) in enumerate(rows):
        a[i] = (BASE + off, issue, nbytes, op)
    return a


def offset_of(prof, ret, ch, di, pl, block, page=0):
    """First byte of a page of a block (stripe = page: consecutive pages of a plane are one full interleave apart)."""
    C, D, P = prof["channels"], prof["dies"], prof["planes"]
    row = block * ret["pages_per_block"] + page
    return (((row * P + pl) * D + di) * C + ch) * PAGE


def block_id(prof, ret, ch, di, pl, block):
    return ((ch * prof["dies"] + di) * prof["planes"] + pl) * ret["blocks_per_plane"] + block


# ---- Arrhenius lifetime and the damage sum ------------------------------------------------------------

def test_lifetime_reference_point_and_shape():
    o, _ = make(RET)
    assert o.retention_lifetime_s(40.0) == 1000.0                       # anchored at the reference condition
    # log L is linear in 1/T: three temperatures equally spaced in 1/T give a geometric sequence
    inv = np.array([1 / 300.0, 1 / 320.0, 1 / 340.0])
    inv[1] = 0.5 * (inv[0] + inv[2])
    L = [o.retention_lifetime_s(1 / x - 273.15) for x in inv]
    assert L[1] ** 2 == pytest.approx(L[0] * L[2], rel=1e-12)
    assert L[0] > L[1] > L[2] > 0
    # with E_a = 1.04 eV the slope -E_a / (k_B T^2) at 328 K is -0.1122 per kelvin: the lifetime halves every 6.2 K
    assert o.retention_lifetime_s(55.0) / o.retention_lifetime_s(55.0 + 6.18) == pytest.approx(2.0, rel=0.02)
    # no activation energy: temperature does not matter
    o2, _ = make(dict(RET, ea_ev=0.0))
    assert o2.retention_lifetime_s(90.0) == 1000.0


def test_damage_reaches_one_after_one_lifetime_at_reference():
    o, _ = make(RET | dict(lead_threshold=10.0))
    nr = 1
    for _ in range(10):
        o.retention_advance(100 * 10**9, np.full(nr, 40.0))             # 10 x 100 s = L_ref
    d = o.retention_blocks()["damage"]
    assert np.allclose(d, 1.0, rtol=1e-12) and d.min() == d.max()
    # acceleration is a plain factor on time
    o2, _ = make(RET | dict(lead_threshold=10.0, accel=4.0))
    o2.retention_advance(250 * 10**9, np.full(nr, 40.0))
    assert np.allclose(o2.retention_blocks()["damage"], 1.0, rtol=1e-12)


def test_eligibility_epoch_is_the_closed_form():
    # lead 0.5, L_ref 1000 s, steps of 60 s at the reference temperature: 0.06 per step, eligible at step 9 (0.54)
    o, _ = make(RET)
    for k in range(1, 10):
        o.retention_advance(60 * 10**9, np.array([40.0]))
        t = o.retention_totals()
        assert t["epoch"] == k
        assert t["waiting_blocks"] == (t["n_blocks"] if k >= 9 else 0)
    b = o.retention_blocks()
    assert (b["epoch"] == 9).all()
    assert o.retention_totals()["planned"] == b["epoch"].size * RET["pages_per_block"]


def test_hotter_region_ages_faster():
    fp = wl.toy_floorplan(16, 48, 8, 4)
    o, prof = make(RET | dict(lead_threshold=1e9), floorplan=fp)
    nr = len(fp["region_kind"])
    temps = np.full(nr, 40.0)
    temps[2 + 3] = 70.0                                                  # channel 3's column
    o.retention_advance(10**9, temps)
    d = o.retention_blocks()["damage"].reshape(prof["channels"], -1)
    assert d[3].min() == d[3].max() and d[0].min() == d[0].max()
    assert d[3][0] / d[0][0] == pytest.approx(o.retention_lifetime_s(40.0) / o.retention_lifetime_s(70.0), rel=1e-12)
    assert d[3][0] > 20 * d[0][0]


def test_region_temperature_from_the_field_is_the_hottest_cell():
    fp = wl.toy_floorplan(16, 48, 8, 4)
    o, prof = make(RET | dict(lead_threshold=1e9), floorplan=fp)
    o2, _ = make(RET | dict(lead_threshold=1e9), floorplan=fp)
    rng = np.random.Generator(np.random.PCG64(5))
    field = 35.0 + 40.0 * rng.random(o.n_cells)
    lib = hbfo.lib()
    lib.hbfo_set_temps(o._h, field.ctypes.data, field.size)
    region = np.asarray(fp["cell_region"]).ravel()
    hottest = np.array([field[region == g].max() for g in range(len(fp["region_kind"]))])
    o.retention_advance(10**9)
    o2.retention_advance(10**9, hottest)
    assert np.array_equal(o.retention_blocks()["damage"], o2.retention_blocks()["damage"])


# ---- the plan ---------------------------------------------------------------------------------------------

def load_example(golden_dir):
    with open(os.path.join(golden_dir, "retention_examples.json")) as f:
        return json.load(f)


def example_context(ex):
    ret = dict(RET, **ex["retention"])
    o, prof = make(ret, **ex["geometry"])
    rows = [(offset_of(prof, ret, b["channel"], b["die"], b["plane"], b["block"]), 0, 64, 0) for b in ex["eligible_blocks"]]
    for b in ex["eligible_blocks"]:
        assert block_id(prof, ret, b["channel"], b["die"], b["plane"], b["block"]) == b["id"]
    o.submit(recs(rows))                                                 # one read each: the disturb limit is 1
    o.retention_advance(0, np.array([40.0]))
    return o, prof, ret


def test_hand_example_plan_claims_commits_decay(golden_dir):
    ex = load_example(golden_dir)
    o, prof, ret = example_context(ex)
    assert o.retention_plan().tolist() == ex["plan"]
    o2, _, _ = example_context(ex)
    # three reads on three idle queues (channel 1: untouched so far)
    rows = [(offset_of(prof, ret, 1, 1, pl, 0), 0, PAGE, 0) for pl in (0, 1)] + [(offset_of(prof, ret, 1, 0, 1, 0), 0, PAGE, 0)]
    _, comp, stall, _, _ = o2.submit(recs(rows))
    assert comp.tolist() == ex["claims"]["completion_first"]
    assert o2.retention_totals()["claimed"] == 3 and o2.retention_totals()["commits"] == 0
    rows = [(offset_of(prof, ret, 1, 1, pl, 0), 1_000_000, PAGE, 0) for pl in (0, 1)]
    _, comp, _, _, _ = o2.submit(recs(rows))
    assert comp.tolist() == ex["claims"]["completion_second"]
    pec = o2.retention_blocks()["pec"]
    assert {str(i): int(v) for i, v in enumerate(pec) if v} == ex["claims"]["pec_after_second"]
    assert o2.retention_plan().tolist() == ex["claims"]["plan_after_second"]
    o2.retention_decay(ex["decay"]["idle_ns"])
    pec = o2.retention_blocks()["pec"]
    assert {str(i): int(v) for i, v in enumerate(pec) if v} == {k: v for k, v in ex["decay"]["pec_after"].items()}
    assert o2.retention_plan().tolist() == ex["decay"]["plan_after"]
    t = o2.retention_totals()
    assert (t["planned"], t["claimed"], t["decayed"], t["commits"]) == (10, 5, 2, 3)
    b = o2.retention_blocks()
    for i in (0, 4, 9):                                                   # committed: counters cleared, no longer waiting
        assert b["damage"][i] == 0.0 and b["disturb"][i] == 0 and b["epoch"][i] == 0
    assert b["epoch"][2] == 1 and b["epoch"][1] == 1


def plan_by_sorting(prof, ret, blocks):
    """Independent formulation: rank within the die by (zone, plane, block, page); within the channel by (that rank,
    die); overall by (rank within the channel, channel)."""
    C, D, P = prof["channels"], prof["dies"], prof["planes"]
    bpp, bpz, ppb = ret["blocks_per_plane"], ret["blocks_per_zone"], ret["pages_per_block"]
    q = []
    for b in blocks:
        k = b % bpp; pl = (b // bpp) % P; di = (b // (bpp * P)) % D; ch = b // (bpp * P * D)
        for pg in range(ppb):
            q.append((ch, di, k // bpz, pl, k, pg, b * ppb + pg))
    q = np.array(q, np.int64).reshape(-1, 7)
    r_die = np.zeros(len(q), np.int64); r_ch = np.zeros(len(q), np.int64)
    for ch in range(C):
        for di in range(D):
            m = np.flatnonzero((q[:, 0] == ch) & (q[:, 1] == di))
            order = m[np.lexsort((q[m, 5], q[m, 4], q[m, 3], q[m, 2]))]
            r_die[order] = np.arange(len(order))
        m = np.flatnonzero(q[:, 0] == ch)
        order = m[np.lexsort((q[m, 1], r_die[m]))]
        r_ch[order] = np.arange(len(order))
    return q[np.lexsort((q[:, 0], r_ch)), 6]


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_plan_order_against_sorting(seed):
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9)
    o, prof = make(ret)
    rng = np.random.Generator(np.random.PCG64([seed, 77]))
    nb = prof["channels"] * prof["dies"] * prof["planes"] * ret["blocks_per_plane"]
    planned = []
    for epoch in range(3):                                               # three epochs: the plan is epoch-major
        free = np.setdiff1d(np.arange(nb), np.array(planned, np.int64))
        pick = np.sort(rng.choice(free, size=int(rng.integers(1, 40)), replace=False))
        if seed == 2 and epoch == 0:
            pick = pick[pick < nb // prof["channels"]]                    # everything on channel 0: no interleave at all
            if pick.size == 0:
                pick = np.array([3])
        rows = []
        for b in pick:
            k = b % ret["blocks_per_plane"]; pl = (b // ret["blocks_per_plane"]) % prof["planes"]
            di = (b // (ret["blocks_per_plane"] * prof["planes"])) % prof["dies"]
            ch = b // (ret["blocks_per_plane"] * prof["planes"] * prof["dies"])
            rows.append((offset_of(prof, ret, ch, di, pl, k, int(rng.integers(0, ret["pages_per_block"]))), 0, 64, 0))
        o.submit(recs(rows))                                             # (these reads also claim what earlier epochs planned)
        o.retention_advance(0, np.array([40.0]))
        plan = o.retention_plan()
        want = plan_by_sorting(prof, ret, pick.tolist())
        assert np.array_equal(plan[len(plan) - len(want):], want)        # the new epoch goes behind everything older
        planned += pick.tolist()
    t = o.retention_totals()
    assert t["planned"] == len(planned) * ret["pages_per_block"] and len(np.unique(plan)) == len(plan) == t["planned"] - t["claimed"]


# ---- claims ----------------------------------------------------------------------------------------------------

def spaced_reads(prof, n, rng, with_natives=False):
    """One-page reads, 1 ms apart (every queue idle again), on random pages; optionally natives mixed in."""
    off = rng.integers(0, wl.GIB // PAGE, n) * PAGE
    a = recs([(int(o), 1_000_000 * (i + 1), 4096, 0) for i, o in enumerate(off)])
    if with_natives:
        nat = rng.random(n) < 0.3
        a["addr"][nat] = 0x1000                                          # below every registered range
    return a


def test_first_claims_go_to_the_first_modeled_accesses_by_index():
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9, pages_per_block=1)
    rng = np.random.Generator(np.random.PCG64(11))
    o, prof = make(ret)
    o.submit(recs([(offset_of(prof, ret, c, 0, 0, 0), 0, 64, 0) for c in range(5)]))
    o.retention_advance(0, np.array([40.0]))
    assert o.retention_totals()["planned"] == 5
    acc = spaced_reads(prof, 40, rng, with_natives=True)
    plain, _ = make()
    _, c0, s0, st0, _ = plain.submit(acc)
    _, c1, s1, st1, _ = o.submit(acc)
    modeled = np.flatnonzero(st1 == 1)
    extra = s1 - s0
    assert np.array_equal(st0, st1)
    assert (extra[modeled[:5]] == 395_000).all() and (extra[modeled[5:]] == 0).all()
    assert (extra[st1 == 0] == 0).all()
    t = o.retention_totals()
    assert t["claimed"] == 5 and t["commits"] == 5 and o.retention_plan().size == 0


def test_all_claiming_batch_equals_a_slower_medium():
    """If every access of a one-page-read stream claims a quantum, the run is that of a medium whose page read
    takes t_read + (t_read + t_prog)."""
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9, pages_per_block=64, blocks_per_plane=64)
    o, prof = make(ret)
    rows = [(offset_of(prof, ret, c, d, 0, 0), 0, 64, 0) for c in range(8) for d in range(4)]
    o.submit(recs(rows))
    o.retention_advance(0, np.array([40.0]))
    debt = o.retention_totals()["planned"]
    w = wl.tiny_uniform(n=2000, seed=4, rho=0.9)
    assert debt >= 2000
    acc = w.acc.copy(); acc["issue_ns"] += 10**8
    slow, _ = make(t_read_ns=20000 + 395000)
    _, c_want, s_want, _, ds_want = slow.submit(acc)
    _, c, s, _, ds = o.submit(acc)
    assert np.array_equal(c, c_want) and np.array_equal(s, s_want)
    assert np.array_equal(ds["busy_ns"], ds_want["busy_ns"])
    assert o.last_result()["service_ns"] == slow.last_result()["service_ns"]


def test_claim_is_thermally_scaled_and_booked_as_energy():
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9, pages_per_block=2)
    o, prof = make(ret)
    o.submit(recs([(0, 0, 64, 0)]))
    o.retention_advance(0, np.array([40.0]))
    lib = hbfo.lib()
    lib.hbfo_force_mode(o._h, 1, 500_000)
    pend0 = np.zeros(o.n_dies, np.int64); lib.hbfo_get_pending_energy(o._h, pend0.ctypes.data, pend0.size)
    off = offset_of(prof, ret, 3, 2, 1, 0)
    _, comp, _, _, ds = o.submit(recs([(off, 10**8, 4096, 0)]))
    assert comp[0] == 10**8 + 790_000 + 40_000 + 171                   # quantum and page read at q = 0.5, then 4 KiB out
    pend = np.zeros(o.n_dies, np.int64); lib.hbfo_get_pending_energy(o._h, pend.ctypes.data, pend.size)
    die = 3 * prof["dies"] + 2
    quantum_pj = (84 + 840) * PAGE
    assert pend[die] - pend0[die] == quantum_pj + 84 * 4096 and (np.delete(pend - pend0, die) == 0).all()
    assert ds["energy_pj"][die] == 84 * 4096 and ds["busy_ns"][die] == 790_000 + 40_000


# ---- disturb, commits, wear, fail-closed -------------------------------------------------------------------------

def test_read_disturb_counts_page_reads_per_block():
    ret = dict(RET, lead_threshold=1e9)
    o, prof = make(ret)
    rng = np.random.Generator(np.random.PCG64(3))
    n = 3000
    off = rng.integers(0, 4096, n) * PAGE + rng.integers(0, 4, n) * 4096
    nbytes = rng.choice([64, 4096, 3 * PAGE], n)
    op = (rng.random(n) < 0.2).astype(np.int64)
    acc = recs([(int(o_), 1000 * i, int(b), int(p)) for i, (o_, b, p) in enumerate(zip(off, nbytes, op))])
    o.submit(acc)
    C, D, P = prof["channels"], prof["dies"], prof["planes"]
    want = np.zeros(C * D * P * ret["blocks_per_plane"], np.int64)
    for o_, b, p in zip(off.tolist(), nbytes.tolist(), op.tolist()):
        if p:
            continue
        u = o_ // PAGE
        ch, di, pl, row = u % C, (u // C) % D, (u // (C * D)) % P, u // (C * D * P)
        blk = ((ch * D + di) * P + pl) * ret["blocks_per_plane"] + (row // ret["pages_per_block"]) % ret["blocks_per_plane"]
        want[blk] += (o_ % PAGE + b + PAGE - 1) // PAGE
    assert np.array_equal(o.retention_blocks()["disturb"], want)


def test_wear_out_after_max_pec_cycles():
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9, pages_per_block=1, max_pec=2)
    o, prof = make(ret)
    for cycle in range(3):
        o.submit(recs([(0, 10**7 * (3 * cycle + 1), 64, 0)]))             # disturbs block 0 (and pays any debt first)
        o.retention_advance(0, np.array([40.0]))
        o.retention_decay(10**6)
    t = o.retention_totals()
    b = o.retention_blocks()
    assert b["pec"][0] == 2 and t["worn_blocks"] == 1 and t["commits"] == 2
    assert b["epoch"][0] == 0 and t["planned"] == 2                       # a worn block is not planned again
    d0 = o.retention_blocks()["damage"][0]
    o.retention_advance(10**9, np.array([40.0]))
    assert o.retention_blocks()["damage"][0] == d0 and o.retention_blocks()["damage"][1] > 0


def test_refused_batch_changes_nothing():
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9)
    o, prof = make(ret)
    o.submit(recs([(0, 0, 64, 0)]))
    o.retention_advance(0, np.array([40.0]))
    before = (o.retention_totals(), o.retention_blocks())
    bad = recs([(PAGE, 10**7, 64, 0), (wl.GIB - 32, 10**7, 64, 0)])      # the second one runs off the end of the range
    rc, *_ = o.submit(bad, check=False)
    assert rc != 0
    after = (o.retention_totals(), o.retention_blocks())
    assert before[0] == after[0]
    for k in before[1]:
        assert np.array_equal(before[1][k], after[1][k])


def test_with_the_paged_submit_every_part_claims_and_disturbs_on_its_own():
    """A 32 KiB read is two parts on two channels (stripe = page).  With two quanta owed both parts claim: each is served
    395,000 + 20,000 ns from 10^6 on its own queue and moves its 16 KiB in 683 ns, so the access ends at 10^6 + 415,683 (as
    one request of two pages it claims once and ends at 10^6 + 395,000 + 40,000 + 1,366).  With one quantum owed only the
    first part claims.  Each part disturbs the block of its own page."""
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9, pages_per_block=2)
    o, prof = make(ret)
    o.submit(recs([(offset_of(prof, ret, 5, 0, 0, 0), 0, 64, 0)]))
    o.retention_advance(0, np.array([40.0]))                              # block (5, 0, 0, 0) is due: two quanta
    row = recs([(offset_of(prof, ret, 0, 0, 0, 0), 10**6, 2 * PAGE, 0)])
    whole, _ = make(ret)
    whole.submit(recs([(offset_of(prof, ret, 5, 0, 0, 0), 0, 64, 0)]))
    whole.retention_advance(0, np.array([40.0]))
    assert whole.submit(row)[1].tolist() == [10**6 + 436_366] and whole.retention_totals()["claimed"] == 1
    _, comp, _, _, ds = o.submit(row, paged=True)
    assert comp.tolist() == [10**6 + 415_683]
    t = o.retention_totals()
    assert t["claimed"] == 2 and t["commits"] == 1
    P = prof["planes"]
    busy = o.busy_until()
    assert busy[(0 * prof["dies"] + 0) * P] == 10**6 + 415_000 and busy[(1 * prof["dies"] + 0) * P] == 10**6 + 415_000
    d = o.retention_blocks()["disturb"]
    assert d[block_id(prof, ret, 0, 0, 0, 0)] == 1 and d[block_id(prof, ret, 1, 0, 0, 0)] == 1
    assert int(ds["busy_ns"].sum()) == 2 * 415_000 and int(ds["n_read"].sum()) == 2
    # one quantum owed: the first part of the list claims, the second does not
    ret1 = dict(ret, pages_per_block=1)
    o1, prof = make(ret1)
    o1.submit(recs([(offset_of(prof, ret1, 5, 0, 0, 0), 0, 64, 0)]))
    o1.retention_advance(0, np.array([40.0]))
    _, comp, _, _, _ = o1.submit(recs([(offset_of(prof, ret1, 0, 0, 0, 0), 10**6, 2 * PAGE, 0)]), paged=True)
    assert comp.tolist() == [10**6 + 415_683] and o1.retention_totals()["claimed"] == 1
    busy = o1.busy_until()
    assert busy[(0 * prof["dies"] + 0) * P] == 10**6 + 415_000 and busy[(1 * prof["dies"] + 0) * P] == 10**6 + 20_000


def test_with_the_channel_bus_claims_lengthen_the_array_stage_only():
    """Two reads on two dies of one channel, both claiming: the arrays finish at 415,000; the bus then moves the
    first read's 16 KiB until 415,683 and the second's until 416,366."""
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9, pages_per_block=2)
    o, prof = make(ret)
    o.enable_channel_bus()
    o.submit(recs([(offset_of(prof, ret, 5, 0, 0, 0), 0, 64, 0)]))
    o.retention_advance(0, np.array([40.0]))
    rows = [(offset_of(prof, ret, 0, 0, 0, 0), 10**6, PAGE, 0), (offset_of(prof, ret, 0, 1, 0, 0), 10**6, PAGE, 0)]
    _, comp, _, _, _ = o.submit(recs(rows))
    assert comp.tolist() == [10**6 + 415_683, 10**6 + 416_366]
    assert o.retention_totals()["claimed"] == 2


def test_with_the_energy_bins_a_claimed_quantum_is_an_event_of_its_own():
    """One claim on an idle queue, bins of 100 us: the quantum (395 us, 15.1 uJ) fills bins 10..13 in proportion to the
    time it spends in each, the read's own 20 us and 344 nJ follow in bin 13/14; nothing goes to the pending totals."""
    ret = dict(RET, disturb_limit=1, lead_threshold=1e9, pages_per_block=1)
    o, prof = make(ret)
    o.enable_energy_bins(100_000, 32)
    o.submit(recs([(0, 0, 64, 0)]))
    o.retention_advance(0, np.array([40.0]))
    first, before = o.energy_bins()
    off = offset_of(prof, ret, 3, 2, 1, 0)
    _, comp, _, _, _ = o.submit(recs([(off, 1_000_000, 4096, 0)]))
    assert comp[0] == 1_000_000 + 395_000 + 20_000 + 171
    first, bins = o.energy_bins()
    die = 3 * prof["dies"] + 2
    got = (bins - before)[:, die]
    quantum_pj, read_pj = (84 + 840) * PAGE, 84 * 4096
    want = np.zeros(32, np.int64)
    for k in range(10, 13):
        want[k] = quantum_pj * 100_000 // 395_000
    want[13] = quantum_pj - 3 * (quantum_pj * 100_000 // 395_000)        # the quantum's last bin takes what is left
    want[13] += read_pj * 5_000 // 20_000                                 # the read's service runs from 1,395,000 to 1,415,000
    want[14] = read_pj - read_pj * 5_000 // 20_000
    assert got.tolist() == want.tolist()
    assert int((bins - before).sum()) == quantum_pj + read_pj
    pend = np.zeros(o.n_dies, np.int64); hbfo.lib().hbfo_get_pending_energy(o._h, pend.ctypes.data, pend.size)
    assert int(pend.sum()) == 0
