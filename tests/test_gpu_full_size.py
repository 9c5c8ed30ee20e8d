"""Parity at the benchmark's full size: the 200 M-access capacity-mode batch, device-resident, in the launch
configuration bench.py times.  Queues are independent, so the oracle is run on sub-streams of whole queues: the
2,048 queues are dealt to as many oracle instances as the host has cores, each serves its own sub-stream (plain
sequential code, one instance per thread), and every completion, stall, per-die total, queue state and summary of the
library is compared with them: all 200 M accesses, on a fresh batch and on a replay (every queue backlogged)."""
import os
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import hbfo
from paper_2609_09800_b200 import workloads as wl

N_FULL = 200_000_000


@pytest.fixture(scope="module")
def full():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    if torch.cuda.get_device_properties(0).total_memory < 60 * (1 << 30):
        pytest.skip("needs a large-memory GPU")
    from paper_2609_09800_b200 import build, hbf
    build.build()
    w = wl.capacity_mode(n=N_FULL)
    from paper_2609_09800_b200.config import fingerprint_streams as fps
    assert fps.sha256_of(w.acc) == fps.recorded()["sha256"]["capacity_mode(200,000,000, seed 0)"]   # the stream every number is quoted on
    u = ((w.acc["addr"] - np.uint64(wl.RANGE_BASE)) >> np.uint64(16)).astype(np.int64)   # 64 KiB stripe units
    queue = (((u % 64) * 8 + (u // 64) % 8) * 4 + (u // 512) % 4).astype(np.int32)
    shards = shards_of(queue, host_workers())
    assert sum(s.size for s in shards) == N_FULL
    return hbf, w, shards, [w.acc[s] for s in shards]


def run_gpu(hbf, ctx, w):
    import torch
    n = w.n
    d_acc = torch.from_numpy(w.acc.view(np.int64).reshape(-1)).cuda()
    d_comp = torch.empty(n, dtype=torch.int64, device="cuda")
    d_stall = torch.empty(n, dtype=torch.int64, device="cuda")
    d_status = torch.empty(n, dtype=torch.uint8, device="cuda")
    d_ds = torch.empty(ctx.n_dies * 6, dtype=torch.int64, device="cuda")
    ws = ctx.workspace(n)
    out = []
    for _ in range(2):                                     # fresh batch, then the same batch on backlogged queues
        assert ctx.submit_batch(d_acc, n, d_comp, d_stall, d_status, d_ds, ws) == 0
        res = ctx.last_result()
        assert res["code"] == 0
        out.append((d_comp.cpu().numpy(), d_stall.cpu().numpy(), d_ds.cpu().numpy().view(hbf.DIE_STATS_DTYPE).copy(),
                    ctx.get_busy_until(), res))
        assert bool((d_status == 1).all())
    del d_acc, d_comp, d_stall, d_status, d_ds
    return out


def host_workers():
    return max(1, min(32, len(os.sched_getaffinity(0))))


def shards_of(queue, groups):
    """Record indices of each group of queues (queue q belongs to group q mod groups), in batch order."""
    grp = (queue % groups).astype(np.int8)
    return [np.flatnonzero(grp == k) for k in range(groups)]


def make_oracle(w, setup=None):
    o = hbfo.Oracle(w.profile)
    for r in w.ranges:
        o.register_range(*r)
    if setup:
        setup(o)
    return o


def compare_shard(o, sub, idx, comp, stall):
    """One oracle instance serves its sub-stream; returns its per-die totals, queue state and summary."""
    _, c_o, s_o, st_o, ds_o = o.submit(sub)
    bad = np.flatnonzero(comp[idx] != c_o)
    assert bad.size == 0, (int(idx[bad[0]]), int(comp[idx[bad[0]]]), int(c_o[bad[0]]), int(bad.size))
    assert np.array_equal(stall[idx], s_o) and (st_o == hbfo.ST_READY).all()
    return ds_o, o.busy_until(), o.last_result()


def check_against_shards(hbf, pool, oracles, subs, shards, comp, stall, ds, busy, res):
    t0 = time.perf_counter()
    outs = list(pool.map(lambda k: compare_shard(oracles[k], subs[k], shards[k], comp, stall), range(len(shards))))
    dt = time.perf_counter() - t0
    ds_sum = np.zeros_like(outs[0][0])
    for f in hbfo.DIE_STATS_DTYPE.names:
        ds_sum[f] = sum(o[0][f] for o in outs)
        assert np.array_equal(ds[f], ds_sum[f]), f
    assert np.array_equal(busy, sum(o[1] for o in outs))     # an instance leaves the queues of the others at zero
    assert res["n_modeled"] == sum(o[2]["n_modeled"] for o in outs) and res["n_native"] == 0
    assert res["modeled_ns"] == sum(o[2]["modeled_ns"] for o in outs)
    assert res["service_ns"] == sum(o[2]["service_ns"] for o in outs)
    assert res["max_completion_ns"] == max(o[2]["max_completion_ns"] for o in outs)
    return dt


@pytest.mark.parametrize("path", ["auto", "sort"])
def test_full_size_batch_against_the_oracle_on_every_queue(full, path):
    hbf, w, shards, subs = full
    ctx = hbf.Context(w.profile)
    for r in w.ranges:
        ctx.register_range(*r)
    ctx.set_path(hbf.PATH_AUTO if path == "auto" else hbf.PATH_SORT)
    runs = run_gpu(hbf, ctx, w)
    issue = w.acc["issue_ns"]
    groups = len(shards)
    oracles = [make_oracle(w) for _ in range(groups)]
    with ThreadPoolExecutor(groups) as pool:
        for step, (comp, stall, ds, busy, res) in enumerate(runs):
            assert np.array_equal(stall, comp - issue)
            dt = check_against_shards(hbf, pool, oracles, subs, shards, comp, stall, ds, busy, res)
            print("\n%s path, pass %d: the oracle served and checked %d accesses on %d threads in %.1f s (%.1f M accesses/s)"
                  % (path, step, N_FULL, groups, dt, N_FULL / dt / 1e6))
    ctx.destroy()


def test_full_size_batch_with_refresh_claims(full):
    """Retention on, in the configuration `bench.py --workload capacity_retention` times: the batch, one epoch that
    makes every block eligible, the batch again with its first 33.5 M accesses claiming one refresh quantum each.
    Claims go to the modeled accesses in index order, so within a sub-stream of whole queues they go to a prefix too:
    every oracle instance serves its sub-stream with exactly that many quanta of debt (made by an epoch of its own and
    trimmed by idle-time decay) and must give the same completions, per-die totals and queue state: all 200 M accesses."""
    import torch
    hbf, w, shards, subs = full
    ret = dict(pages_per_block=256, blocks_per_plane=64, blocks_per_zone=8, max_pec=3000, disturb_limit=1,
               l_ref_s=3.15e7, t_ref_c=40.0, ea_ev=1.04, accel=1.0, lead_threshold=0.8)
    ctx = hbf.Context(w.profile)
    for r in w.ranges:
        ctx.register_range(*r)
    ctx.enable_retention(**ret)
    n = w.n
    d_acc = torch.from_numpy(w.acc.view(np.int64).reshape(-1)).cuda()
    d_comp = torch.empty(n, dtype=torch.int64, device="cuda"); d_stall = torch.empty_like(d_comp)
    d_ds = torch.empty(ctx.n_dies * 6, dtype=torch.int64, device="cuda")
    ws = ctx.workspace(n)
    assert ctx.submit_batch(d_acc, n, d_comp, d_stall, None, d_ds, ws) == 0
    assert ctx.last_result()["code"] == 0 and ctx.retention_totals()["claimed"] == 0
    ctx.retention_advance(10**9, np.array([60.0]))
    debt = ctx.retention_totals()["planned"]
    assert debt == 131072 * 256                               # every block was read at least once
    assert ctx.submit_batch(d_acc, n, d_comp, d_stall, None, d_ds, ws) == 0
    res = ctx.last_result()
    comp = d_comp.cpu().numpy(); ds = d_ds.cpu().numpy().view(hbf.DIE_STATS_DTYPE).copy(); busy = ctx.get_busy_until()
    tot = ctx.retention_totals()
    assert res["code"] == 0 and tot["claimed"] == debt and tot["commits"] == 131072 and tot["waiting_blocks"] == 0
    npages = np.maximum(1, w.acc["bytes"].astype(np.int64) >> 14)
    assert res["service_ns"] == int(npages.sum()) * 20000 + debt * 395000 == int(ds["busy_ns"].sum())
    assert int(ctx.retention_blocks()["pec"].sum()) == 131072
    quantum_pj = (84 + 840) * 16384
    read_pj = 2 * 84 * int(np.maximum(w.acc["bytes"], 64).astype(np.int64).sum())          # two batches of reads
    assert int(ctx.get_pending_energy().sum()) == read_pj + debt * quantum_pj
    del d_acc, d_comp, d_stall, d_ds
    stall = comp - w.acc["issue_ns"]

    def with_debt(k, sub):
        def setup(o):                                         # every block eligible after one epoch; all but k quanta drained
            o.enable_retention(**dict(ret, disturb_limit=0, lead_threshold=1e-9))
            o.submit(sub)
            o.retention_advance(10**9, np.array([60.0]))
            assert o.retention_totals()["planned"] == debt
            o.retention_decay((debt - k) * 395000)
            assert o.retention_totals()["planned"] - o.retention_totals()["decayed"] == k
        return setup

    ks = [int(np.count_nonzero(idx < debt)) for idx in shards]   # every access is modeled: the claim limit is the debt itself
    assert sum(ks) == debt
    with ThreadPoolExecutor(len(shards)) as pool:
        oracles = list(pool.map(lambda j: make_oracle(w, with_debt(ks[j], subs[j])), range(len(shards))))
        outs = list(pool.map(lambda j: compare_shard(oracles[j], subs[j], shards[j], comp, stall), range(len(shards))))
    for f in ("busy_ns", "bytes_read", "n_read", "energy_pj"):
        assert np.array_equal(ds[f], sum(o[0][f] for o in outs)), f
    assert np.array_equal(busy, sum(o[1] for o in outs))
    assert res["service_ns"] == sum(o[2]["service_ns"] for o in outs)
    assert ctx.last_result()["modeled_ns"] == sum(o[2]["modeled_ns"] for o in outs)
    ctx.destroy()


def test_tile_sizes_from_measurements_leave_every_result_as_it_was():
    """A batch that fills one wave of the device (two tiles per SM) leaves each tile's time; the next batches cut their tiles
    in proportion to the measured rates.  Results must not move: three batches with the measurements on (fixed sizes,
    then sizes from one and from two measurements) against the same batch with them off, and against the oracle."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_09800_b200 import build, hbf
    build.build()
    n = 24_000_123
    w = wl.capacity_mode(n=n, seed=5)
    d_acc = torch.from_numpy(w.acc.view(np.int64).reshape(-1)).cuda()
    d_comp = torch.empty(n, dtype=torch.int64, device="cuda"); d_stall = torch.empty_like(d_comp)
    d_status = torch.empty(n, dtype=torch.uint8, device="cuda")
    outs, lens = [], []
    for on in (False, True):
        ctx = hbf.Context(w.profile)
        for r in w.ranges:
            ctx.register_range(*r)
        ctx.set_tile_balance(on)
        d_ds = torch.empty(ctx.n_dies * 6, dtype=torch.int64, device="cuda")
        ws = ctx.workspace(n)
        for k in range(3 if on else 1):
            ctx.reset()
            assert ctx.submit_batch(d_acc, n, d_comp, d_stall, d_status, d_ds, ws) == 0 and ctx.last_result()["code"] == 0
            outs.append((d_comp.cpu().numpy(), d_stall.cpu().numpy(), d_ds.cpu().numpy().copy(), ctx.get_busy_until(), ctx.last_result()))
            rec, ns = ctx.tile_times()
            if on:
                sms = torch.cuda.get_device_properties(0).multi_processor_count
                assert rec.size == 2 * sms and int(rec.astype(np.int64).sum()) == n and (ns > 0).sum() >= rec.size - 4
                lens.append(rec.copy())
            else:
                assert rec.size == 0
        ctx.destroy()
    assert np.unique(lens[0]).size <= 6                       # the two nominal sizes, give or take a quantum, and the ragged last tile
    assert np.unique(lens[2]).size > 8 and not np.array_equal(lens[1], lens[0])      # sized tile by tile
    base = outs[0]
    for o in outs[1:]:
        assert np.array_equal(o[0], base[0]) and np.array_equal(o[1], base[1]) and np.array_equal(o[2], base[2])
        assert np.array_equal(o[3], base[3]) and o[4] == base[4]
    orc = hbfo.Oracle(w.profile)
    for r in w.ranges:
        orc.register_range(*r)
    _, c_o, s_o, _, ds_o = orc.submit(w.acc)
    assert np.array_equal(base[0], c_o) and np.array_equal(base[1], s_o)
    assert np.array_equal(base[3], orc.busy_until())


@pytest.mark.parametrize("which", ["decode_weights", "prefix_kv"])
def test_serving_configurations_at_full_size_element_by_element(which):
    """The 21 M-access decode-weight stream and the 28 M-access prefix-KV stream (the two serving configurations),
    device-resident and in one batch each as the bench would submit them: the oracle serves them whole in a few
    seconds, so every completion, stall, status, per-die statistic and queue state is compared; then the same batch
    again on the queues it left backlogged."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_09800_b200 import build, hbf
    build.build()
    w = wl.decode_weights() if which == "decode_weights" else wl.prefix_kv()
    from paper_2609_09800_b200.config import fingerprint_streams as fps
    assert fps.sha256_of(w.acc) == fps.recorded()["sha256"]["decode_weights(256 tokens, seed 0)" if which == "decode_weights" else "prefix_kv(seed 0)"]
    g, o = hbf.Context(w.profile), hbfo.Oracle(w.profile)
    for r in w.ranges:
        g.register_range(*r); o.register_range(*r)
    n = w.n
    d_acc = torch.from_numpy(w.acc.view(np.int64).reshape(-1)).cuda()
    d_comp = torch.empty(n, dtype=torch.int64, device="cuda"); d_stall = torch.empty_like(d_comp)
    d_status = torch.empty(n, dtype=torch.uint8, device="cuda")
    d_ds = torch.empty(g.n_dies * 6, dtype=torch.int64, device="cuda")
    ws = g.workspace(n)
    for _ in range(2):
        assert g.submit_batch(d_acc, n, d_comp, d_stall, d_status, d_ds, ws) == 0
        _, c_o, s_o, st_o, ds_o = o.submit(w.acc)
        assert g.last_result() == o.last_result()
        c_g = d_comp.cpu().numpy()
        bad = np.flatnonzero(c_g != c_o)
        assert bad.size == 0, "first mismatch at %d: gpu %d oracle %d (%d mismatches)" % (bad[0], c_g[bad[0]], c_o[bad[0]], bad.size)
        assert np.array_equal(d_stall.cpu().numpy(), s_o) and np.array_equal(d_status.cpu().numpy(), st_o)
        ds_g = d_ds.cpu().numpy().view(hbf.DIE_STATS_DTYPE)
        for k in hbfo.DIE_STATS_DTYPE.names:
            assert np.array_equal(ds_g[k], ds_o[k]), k
        assert np.array_equal(g.get_busy_until(), o.busy_until())
