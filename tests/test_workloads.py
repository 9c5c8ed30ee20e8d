"""The seeded input generators: counts, ranges, ordering and determinism."""
import numpy as np

from paper_2609_09800_b200 import workloads as wl


def in_ranges(w):
    ok = np.zeros(w.n, bool)
    for base, length, *_ in w.ranges:
        ok |= (w.acc["addr"] >= base) & (w.acc["addr"] + w.acc["bytes"] <= base + length)
    return ok


def test_model_shapes_match_the_paper_expert_set():
    assert wl.N_LAYERS * wl.N_EXPERTS * wl.EXPERT_BYTES == 54 * wl.GIB
    assert wl.WEIGHT_BYTES == 59_793_997_824 and wl.KV_BYTES == 768 * wl.MIB
    assert wl.KV_OFFSET + wl.KV_BYTES <= wl.SERVING_RANGE and wl.WEIGHT_BYTES <= wl.KV_OFFSET


def test_tiny_uniform():
    w = wl.tiny_uniform()
    assert w.n == 65536 and (w.acc["bytes"] == 4096).all() and not w.acc["flags"].any()
    assert in_ranges(w).all() and (np.diff(w.acc["issue_ns"]) >= 0).all()
    assert abs(np.diff(w.acc["issue_ns"]).mean() - 625.0) < 10
    assert np.array_equal(w.acc, wl.tiny_uniform().acc)
    assert not np.array_equal(w.acc, wl.tiny_uniform(seed=1).acc)


def test_decode_weights_counts():
    w = wl.decode_weights(tokens=3)
    assert w.n == 3 * 82944 and (w.acc["bytes"] == 65536).all()
    assert in_ranges(w).all() and (np.diff(w.acc["issue_ns"]) >= 0).all()
    off = (w.acc["addr"] - wl.RANGE_BASE).astype(np.int64)
    assert (off % 65536 == 0).all() and off.max() < wl.WEIGHT_BYTES
    per_layer = off[:82944].reshape(48, 576 + 8 * 144)
    assert (per_layer // wl.LAYER_BYTES == np.arange(48)[:, None]).all()
    experts = (per_layer[:, 576::144] % wl.LAYER_BYTES - wl.ATTN_BYTES) // wl.EXPERT_BYTES
    assert all(len(set(r)) == 8 for r in experts.tolist())               # top-8 without replacement


def test_prefix_kv_small():
    w = wl.prefix_kv(epochs=1, steps=1, batch=4, kv_tokens=256, layers=2)
    prog = w.acc["flags"] == 1
    assert prog.sum() == 2 * 256 * 2048 // 4096 and (w.acc["bytes"][prog] == 4096).all()
    assert in_ranges(w).all() and (np.diff(w.acc["issue_ns"]) >= 0).all()
    assert (w.acc["addr"][prog] - wl.RANGE_BASE >= wl.KV_OFFSET).all()


def test_capacity_chunks_are_deterministic_and_sorted():
    w = wl.capacity_mode(n=300_000)
    parts = np.concatenate(list(wl.capacity_chunks(n=300_000, workers=1)))
    assert np.array_equal(w.acc, parts)
    assert in_ranges(w).all() and (np.diff(w.acc["issue_ns"]) >= 0).all()
    sz = w.acc["bytes"].astype(np.int64)
    assert set(np.unique(sz).tolist()) == {1 << k for k in range(7, 17)}
    off = (w.acc["addr"] - wl.RANGE_BASE).astype(np.int64) % wl.CAPACITY_SLOT
    assert (off % sz == 0).all() and (off + sz <= wl.WEIGHT_BYTES).all()


def test_timed_batches_cover_the_stream_and_repeat():
    w = wl.tiny_uniform(5000)
    span = int(w.acc["issue_ns"][-1]) + 1
    horizon = 2 * span + 12345
    got = list(wl.timed_batches(w, horizon, 1_000_000))
    allrec = np.concatenate([b for _, b in got])
    assert (np.diff(allrec["issue_ns"]) >= 0).all()
    for k, b in got:
        assert ((b["issue_ns"] >= k * 1_000_000) & (b["issue_ns"] < (k + 1) * 1_000_000)).all()
    assert np.array_equal(allrec[:5000], w.acc)
    assert np.array_equal(allrec["addr"][5000:10000], w.acc["addr"])
    assert (allrec["issue_ns"][5000:10000] == w.acc["issue_ns"] + span).all()


def test_floorplans():
    fp = wl.package_floorplan()
    assert fp["grid_h"] == fp["grid_w"] == 128 and len(fp["region_kind"]) == 63 and len(fp["die_region"]) == 256
    region = fp["cell_region"].reshape(128, 128)
    assert (region[8:24, 32:48] == 0).all() and (np.bincount(region[region >= 31])[31:] == 72).all()
    assert abs(float(fp["ext_power_w"].sum()) - (86.6 + 24.0)) < 1e-4 and abs(float(fp["region_idle_w"].sum()) - 10.0) < 1e-6
    assert (fp["cell_Gx"].reshape(128, 128)[:, -1] == 0).all() and (fp["cell_Gy"].reshape(128, 128)[-1] == 0).all()
    # unlike neighbours: series half cells
    gx = fp["cell_Gx"].reshape(128, 128)
    assert abs(gx[10, 31] - 2 * 0.03 * 0.075 / 0.105) < 1e-7


def test_stream_fingerprints():
    """The committed SHA-256 of every stream small enough for this box (the two largest are checked where they are used, on
    the GPU machine): a numpy release or an edit that reshuffles a stream fails here, and the file names the numpy it was made with."""
    from paper_2609_09800_b200.config import fingerprint_streams as fps
    rec = fps.recorded()
    assert set(rec["sha256"]) == set(fps.STREAMS) and rec["numpy"].split(".")[0] == np.__version__.split(".")[0]
    got = fps.compute(cheap_only=True)
    assert len(got) >= 5
    for name, sha in got.items():
        assert rec["sha256"][name] == sha, name
