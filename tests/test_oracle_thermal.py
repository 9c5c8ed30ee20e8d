"""Pins of the CPU oracle's thermal step: the paper's printed power figure, the lumped closed form,
steady state against a direct sparse solve, energy balance, superposition and reciprocity, and the
throttle state machine."""
import json
import os

import numpy as np
import pytest
import scipy.sparse as sp
import scipy.sparse.linalg as spla

from oracle import hbfo
from paper_2609_09800_b200 import workloads as wl


def single_node_plan(n_dies, C=1000.0, Gs=1.0, idle=5.0):
    return dict(grid_h=1, grid_w=1, cell_C=[C], cell_Gx=[0.0], cell_Gy=[0.0], cell_Gsink=[Gs],
                cell_region=[0], die_region=[0] * n_dies, region_kind=[wl.KIND_HBF], region_idle_w=[idle])


def uniform_plan(h, w, n_dies, C=2e-4, g=0.05, Gs=2e-4, idle=0.0):
    Gx = np.full((h, w), g); Gx[:, -1] = 0
    Gy = np.full((h, w), g); Gy[-1, :] = 0
    return dict(grid_h=h, grid_w=w, cell_C=np.full(h * w, C), cell_Gx=Gx.ravel(), cell_Gy=Gy.ravel(),
                cell_Gsink=np.full(h * w, Gs), cell_region=np.zeros(h * w, np.int32), die_region=[0] * n_dies,
                region_kind=[wl.KIND_HBF], region_idle_w=[idle])


def conductance_matrix(fp):
    """L_G + diag(G_sink) assembled edge by edge (independent of the oracle's stencil loop)."""
    H, W = fp["grid_h"], fp["grid_w"]
    Gx = np.asarray(fp["cell_Gx"], np.float64).reshape(H, W)
    Gy = np.asarray(fp["cell_Gy"], np.float64).reshape(H, W)
    idx = np.arange(H * W).reshape(H, W)
    rows, cols, vals = [], [], []

    def edge(i, j, g):
        rows.extend([i, j, i, j]); cols.extend([i, j, j, i]); vals.extend([g, g, -g, -g])
    for y in range(H):
        for x in range(W):
            if x + 1 < W:
                edge(idx[y, x], idx[y, x + 1], Gx[y, x])
            if y + 1 < H:
                edge(idx[y, x], idx[y + 1, x], Gy[y, x])
    A = sp.coo_matrix((vals, (rows, cols)), shape=(H * W, H * W)).tocsc()
    return A + sp.diags(np.asarray(fp["cell_Gsink"], np.float64))


def cell_power(fp, ext, die_w=None):
    region = np.asarray(fp["cell_region"])
    pr = np.asarray(fp["region_idle_w"], np.float64) + np.asarray(ext, np.float64)
    if die_w is not None:
        np.add.at(pr, np.asarray(fp["die_region"]), die_w)
    cnt = np.bincount(region[region >= 0], minlength=pr.shape[0])
    return np.where(region >= 0, pr[np.maximum(region, 0)] / np.maximum(cnt[np.maximum(region, 0)], 1), 0.0)


def test_paper_read_power_37_256_w(golden_dir):
    with open(os.path.join(golden_dir, "paper_values.json")) as f:
        pv = json.load(f)["hbf_read_power"]
    prof = wl.load_profile("nominal", channels=16, dies=8, planes=1, page_bytes=16384, stripe_bytes=65536, n_sub=1)
    assert prof["e_byte_read_pj"] * 1e-12 == pytest.approx(pv["joule_per_byte"], rel=1e-12)
    o = hbfo.Oracle(prof, single_node_plan(128, idle=pv["idle_w"]))
    o.register_range(wl.RANGE_BASE, 1 << 40)
    n = int(pv["bytes_per_s"]) // 65536
    assert n * 65536 == int(pv["bytes_per_s"])
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = wl.RANGE_BASE + np.arange(n, dtype=np.uint64) * np.uint64(65536)
    acc["bytes"] = 65536
    _, _, _, _, ds = o.submit(acc)
    assert int(ds["bytes_read"].sum()) == int(pv["bytes_per_s"])
    hot, _ = o.thermal_step(1_000_000_000)                  # one 1 s window, one Euler substep
    # one node, C = 1000 J/K, starting at ambient: the rise after one step is dt/C * P
    assert (hot[0] - prof["ambient_c"]) * 1000.0 == pytest.approx(pv["power_w"], abs=1e-9)
    assert not o.pending_energy().any()                     # the window's energy is consumed


def test_field_starts_at_ambient():
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])
    o = hbfo.Oracle(prof, wl.toy_floorplan(12, 20, 8, 4))
    assert (o.temps() == 35.0).all()


def test_lumped_closed_form():
    # uniform power and constants: no lateral flow, every cell follows (P/G)(1 - (1 - dt G/C)^n)
    h, w = 6, 9
    C, Gs = float(np.float32(2e-4)), float(np.float32(3e-4))       # the floorplan arrays are float32
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"], n_sub=8)
    o = hbfo.Oracle(prof, uniform_plan(h, w, 32, C=C, Gs=Gs, idle=0.0))
    p_total = 27.0 / 2048.0
    n = 0
    for step in range(5):
        _, T = o.thermal_step(800_000, [p_total], want_temps=True)
        n += 8
        want = (p_total / (h * w) / Gs) * (1 - (1 - 1e-4 * Gs / C) ** n)
        assert np.allclose(T - 35.0, want, rtol=0, atol=1e-13)


def test_euler_limit_and_unstable_step_is_refused():
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"], n_sub=1)
    fp = uniform_plan(4, 4, 32, C=2e-4, g=0.05, Gs=2e-4)
    o = hbfo.Oracle(prof, fp)
    lim = 2e-4 / (4 * 0.05 + 2e-4) * 1e9
    assert o.euler_limit_ns() == pytest.approx(lim, rel=1e-6)
    o.thermal_step(int(lim) - 1, [0.0])
    with pytest.raises(hbfo.OracleError):
        o.thermal_step(int(lim) + 2, [0.0])


def test_steady_state_matches_direct_solve():
    fp = wl.toy_floorplan(16, 24, 8, 4, seed=3)
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"], n_sub=2000)
    o = hbfo.Oracle(prof, fp)
    A = conductance_matrix(fp)
    theta = spla.spsolve(A, cell_power(fp, fp["ext_power_w"]))
    dt = int(0.9 * o.euler_limit_ns() * 2000)
    for _ in range(60):
        _, T = o.thermal_step(dt, fp["ext_power_w"], want_temps=True)
    assert np.abs(T - 35.0 - theta).max() < 1e-7 * max(1.0, theta.max())
    # and the solve is a fixed point of one more step, whatever the step length
    o.set_temps(35.0 + theta)
    _, T2 = o.thermal_step(dt // 7, fp["ext_power_w"], want_temps=True)
    assert np.abs(T2 - 35.0 - theta).max() < 1e-9


def test_energy_balance_per_substep():
    fp = wl.toy_floorplan(10, 20, 8, 4, seed=1)
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"], n_sub=1)
    o = hbfo.Oracle(prof, fp)
    C = np.asarray(fp["cell_C"], np.float64); Gs = np.asarray(fp["cell_Gsink"], np.float64)
    P = cell_power(fp, fp["ext_power_w"])
    dt = int(0.5 * o.euler_limit_ns())
    T0 = o.temps()
    for _ in range(50):
        _, T1 = o.thermal_step(dt, fp["ext_power_w"], want_temps=True)
        lhs = (C * (T1 - T0)).sum()
        rhs = dt * 1e-9 * (P.sum() - (Gs * (T0 - 35.0)).sum())       # lateral flows cancel pairwise
        assert lhs == pytest.approx(rhs, rel=1e-9)
        T0 = T1


def _point_source_plan(h, w, cells):
    fp = wl.toy_floorplan(h, w, 8, 4, seed=2)
    region = -np.ones(h * w, np.int32)
    for k, c in enumerate(cells):
        region[c] = k
    fp.update(cell_region=region, region_kind=[wl.KIND_HBF] * len(cells), region_idle_w=[0.0] * len(cells),
              die_region=[0] * 32)
    return fp


def test_superposition_and_reciprocity():
    h, w = 10, 20
    i, j = 2 * w + 3, 7 * w + 14
    fp = _point_source_plan(h, w, [i, j])
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"], n_sub=64)

    def run(ext):
        o = hbfo.Oracle(prof, fp)
        for _ in range(20):
            _, T = o.thermal_step(int(0.8 * o.euler_limit_ns() * 64), ext, want_temps=True)
        return T - 35.0
    a, b, ab = run([1.0, 0.0]), run([0.0, 1.0]), run([2.0, 3.0])
    assert np.allclose(ab, 2 * a + 3 * b, rtol=1e-10, atol=1e-14)         # linear operator
    assert a[j] == pytest.approx(b[i], rel=1e-10)                         # R_ij = R_ji, also in the transient
    assert a[i] > a[j] > 0


def test_die_energy_reaches_its_region():
    fp = wl.toy_floorplan(10, 20, 8, 4, seed=1)
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"], n_sub=1)
    o = hbfo.Oracle(prof, fp)
    o.register_range(wl.RANGE_BASE, wl.GIB)
    acc = np.zeros(64, hbfo.ACCESS_DTYPE)
    acc["addr"] = wl.RANGE_BASE + 3 * 16384             # stripe unit 3 -> channel 3
    acc["bytes"] = 16384
    o.submit(acc)
    dt = int(0.5 * o.euler_limit_ns())
    _, T = o.thermal_step(dt, np.zeros(len(fp["region_kind"])), want_temps=True)
    die_w = np.zeros(32); die_w[3 * 4 + 0] = 64 * 16384 * 84e-12 / (dt * 1e-9)
    want = dt * 1e-9 / np.asarray(fp["cell_C"], np.float64) * cell_power(fp, np.zeros(len(fp["region_kind"])), die_w)
    assert np.allclose(T - 35.0, want, rtol=1e-12, atol=0)
    region = np.asarray(fp["cell_region"])
    assert (T[region == 2 + 3] > T[region == 2 + 4].max()).all()


# ---- throttle state machine -------------------------------------------------------------------------

N, L, S, X = hbfo.MODE_NORMAL, hbfo.MODE_LIGHT, hbfo.MODE_SEVERE, hbfo.MODE_SHUTDOWN


def test_state_machine_table():
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"])        # 80 / 85 / 95 / 105
    o = hbfo.Oracle(prof, wl.toy_floorplan(8, 20, 8, 4))
    table = [  # (mode, T_hot in mK, next)
        (N, 84999, N), (N, 85000, L), (N, 94999, L), (N, 95000, S), (N, 105000, X),
        (L, 80001, L), (L, 80000, N), (L, 94999, L), (L, 95000, S), (L, 105000, X),
        (S, 95000, S), (S, 85001, S), (S, 85000, L), (S, 80001, L), (S, 80000, N), (S, 104999, S), (S, 105000, X),
        (X, 20000, X), (X, 200000, X),
    ]
    for mode, t, want in table:
        assert o.next_mode(mode, t) == want, (mode, t)
    assert hbfo.quantise_mk(84.9995) == 85000 and hbfo.quantise_mk(84.99949) == 84999   # round half up
    assert hbfo.quantise_mk(-0.0005) == 0 and hbfo.quantise_mk(-0.00051) == -1


def test_controller_follows_the_hotspot_with_hysteresis():
    prof = wl.load_profile("nominal", channels=1, dies=1, planes=1, page_bytes=16384, stripe_bytes=16384, n_sub=1)
    o = hbfo.Oracle(prof, single_node_plan(1, C=1.0, Gs=1.0, idle=0.0))
    o.register_range(wl.RANGE_BASE, wl.GIB)
    a = np.zeros(1, hbfo.ACCESS_DTYPE); a["addr"] = wl.RANGE_BASE; a["bytes"] = 4096
    seen = []
    # one node with G = 1 W/K: steady rise = P; drive the hotspot up and back down with the external power
    for p in [40, 51, 51, 61, 61, 52, 48, 46, 44, 71, 71, 30]:
        for _ in range(40):
            hot, _ = o.thermal_step(500_000_000, [float(p)])
        mode, q = o.mode()
        seen.append((p, mode, q))
        rc = o.submit(a, check=False)[0]
        assert rc == {N: 0, L: 0, S: hbfo.E_THROTTLED, X: hbfo.E_LINK_SHUTDOWN}[mode]
    assert [m for _, m, _ in seen] == [N, L, L, S, S, S, L, L, N, X, X, X]
    assert all(q == (800000 if m == L else 1000000) for _, m, q in seen[:3])


def test_thermal_disabled_without_floorplan():
    o = hbfo.Oracle(wl.load_profile("nominal", **wl.GEOMETRY["tiny"]))
    with pytest.raises(hbfo.OracleError):
        o.thermal_step(1000)
