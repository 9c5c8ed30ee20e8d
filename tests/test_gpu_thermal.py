"""Parity of the CUDA thermal step (float32 + compensation) with the float64 CPU oracle: temperatures
within 1e-3 K max-abs, mode / service-fraction traces equal (a threshold tie is allowed only when the
oracle's hotspot sits within 2e-3 K of a threshold)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import hbfo
from paper_2609_09800_b200 import workloads as wl

TOL_K = 1e-3


@pytest.fixture(scope="module")
def hbf():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_09800_b200 import build, hbf as mod
    build.build()
    return mod


def pair(hbf, profile, fp, ranges=()):
    g = hbf.Context(profile, fp)
    o = hbfo.Oracle(profile, fp)
    for r in ranges:
        g.register_range(*r); o.register_range(*r)
    return g, o


def near_threshold(prof, t):
    return min(abs(t - prof[k]) for k in ("rtt_c", "ltt_c", "stt_c", "shutdown_c")) < 2e-3


def step_both(hbf, g, o, prof, dt, ext, want_temps=True):
    import torch
    d_T = torch.empty(g.n_cells, dtype=torch.float32, device="cuda") if want_temps else None
    hot_g = g.thermal_step(dt, ext, d_T)
    hot_o, T_o = o.thermal_step(dt, ext, want_temps=want_temps)
    assert np.abs(hot_g.astype(np.float64) - hot_o).max() < TOL_K
    if want_temps:
        T_g = d_T.cpu().numpy().astype(np.float64)
        assert np.abs(T_g - T_o).max() < TOL_K
    mg, mo = g.get_mode(), o.mode()
    if mg != mo:
        assert near_threshold(prof, hot_o[0]), (mg, mo, hot_o)
        o.force_mode(*mg)                                   # threshold tie: follow the GPU and go on
    return hot_g, hot_o


def test_field_starts_at_ambient(hbf):
    prof = wl.load_profile("nominal", **wl.GEOMETRY["serving"])
    g, _ = pair(hbf, prof, wl.package_floorplan())
    assert (g.get_temps() == np.float32(35.0)).all()
    assert g.euler_limit_ns() == pytest.approx(hbfo.Oracle(prof, wl.package_floorplan()).euler_limit_ns(), rel=1e-12)


def test_package_floorplan_coupled_run(hbf):
    """Config-5 shape at reduced length: 1 ms batches of the prefix-KV stream, each followed by a
    thermal step on the 128x128 package grid; every completion, stat, temperature and mode compared."""
    w = wl.prefix_kv(epochs=1, steps=1, batch=64, kv_tokens=8192, layers=3)
    fp = wl.package_floorplan()
    g, o = pair(hbf, w.profile, fp, w.ranges)
    ext = fp["ext_power_w"]
    n_steps = 0
    for k, acc in wl.timed_batches(w, 400_000_000):
        rc_o, c_o, s_o, _, ds_o = o.submit(acc)
        rc_g, c_g, s_g, _, ds_g = g.submit_host(acc)
        assert np.array_equal(c_g, c_o) and np.array_equal(s_g, s_o)
        assert np.array_equal(ds_g["energy_pj"], ds_o["energy_pj"])
        step_both(hbf, g, o, w.profile, 1_000_000, ext, want_temps=(k % 50 == 49))
        n_steps += 1
    assert n_steps == 400
    hot_g, hot_o = step_both(hbf, g, o, w.profile, 1_000_000, ext)
    assert hot_o[0] > 36.0 and hot_o[2] > 36.0                # the package actually heats up


def test_long_run_stays_within_tolerance(hbf):
    """Many substeps with constant power: the float32 state with compensation must track float64."""
    fp = wl.package_floorplan()
    prof = wl.load_profile("nominal", **wl.GEOMETRY["serving"], n_sub=64)
    g, o = pair(hbf, prof, fp)
    ext = fp["ext_power_w"].copy()
    ext[31:] = 16.5 / 16                                      # with 5 W idle: 21.5 W per HBF stack, the config-5 load
    dt = int(0.9 * o.euler_limit_ns() * 64)
    for k in range(400):                                      # 25,600 substeps, ~3.8 s of simulated time
        step_both(hbf, g, o, prof, dt, ext, want_temps=(k % 100 == 99))
    assert g.get_mode()[0] >= hbf.MODE_LIGHT                  # crossed the light threshold on the way up


@pytest.mark.parametrize("shape", [(17, 45), (8, 20), (33, 64), (3, 40), (130, 131)])
def test_odd_grids(hbf, shape):
    h, w_ = shape
    fp = wl.toy_floorplan(h, w_, 8, 4, seed=h)
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"], n_sub=7)
    g, o = pair(hbf, prof, fp)
    dt = int(0.7 * o.euler_limit_ns() * 7)
    for k in range(60):
        step_both(hbf, g, o, prof, dt, fp["ext_power_w"] * (1 + (k % 3)))


def test_controller_trace_with_hysteresis(hbf):
    prof = wl.load_profile("nominal", channels=1, dies=1, planes=1, page_bytes=16384, stripe_bytes=16384, n_sub=1)
    fp = dict(grid_h=1, grid_w=1, cell_C=[1.0], cell_Gx=[0.0], cell_Gy=[0.0], cell_Gsink=[1.0], cell_region=[0],
              die_region=[0], region_kind=[wl.KIND_HBF], region_idle_w=[0.0])
    g, o = pair(hbf, prof, fp, [(wl.RANGE_BASE, wl.GIB, 3, 0, 0, 0)])
    a = np.zeros(1, hbfo.ACCESS_DTYPE); a["addr"] = wl.RANGE_BASE; a["bytes"] = 4096
    trace = []
    for p in [40, 51, 51, 61, 61, 52, 48, 46, 44, 71, 71, 30]:
        for _ in range(40):
            step_both(hbf, g, o, prof, 500_000_000, [float(p)])
        mode, q = g.get_mode()
        trace.append(mode)
        rc_g = g.submit_host(a, check=False)[0]
        rc_o = o.submit(a, check=False)[0]
        assert rc_g == rc_o
    N, L, S, X = hbf.MODE_NORMAL, hbf.MODE_LIGHT, hbf.MODE_SEVERE, hbf.MODE_SHUTDOWN
    assert trace == [N, L, L, S, S, S, L, L, N, X, X, X]


def test_unstable_step_and_bad_arguments(hbf):
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"], n_sub=1)
    fp = wl.toy_floorplan(8, 20, 8, 4)
    g, o = pair(hbf, prof, fp)
    with pytest.raises(hbf.HbfError):
        g.thermal_step(int(o.euler_limit_ns()) + 10, fp["ext_power_w"])
    with pytest.raises(hbf.HbfError):
        g.thermal_step(1000, fp["ext_power_w"][:3])
    g2 = hbf.Context(prof)
    with pytest.raises(hbf.HbfError):
        g2.thermal_step(1000)


def test_reset_and_state_round_trip(hbf):
    fp = wl.toy_floorplan(12, 24, 8, 4, seed=2)
    prof = wl.load_profile("nominal", **wl.GEOMETRY["tiny"], n_sub=4)
    g, o = pair(hbf, prof, fp)
    dt = int(0.5 * o.euler_limit_ns() * 4)
    for _ in range(25):
        step_both(hbf, g, o, prof, dt, fp["ext_power_w"])
    blob = g.get_state()
    T = g.get_temps()
    g.reset()
    assert (g.get_temps() == np.float32(35.0)).all()
    g.set_state(blob)
    assert np.array_equal(g.get_temps(), T)
    for _ in range(25):
        step_both(hbf, g, o, prof, dt, fp["ext_power_w"])


@pytest.mark.parametrize("shape", [(128, 128), (17, 45), (3, 40), (130, 131), (64, 64)])
def test_cluster_step_equals_per_substep_launches(hbf, shape):
    """The one-launch cluster kernel and the launch-per-substep kernels perform the same arithmetic."""
    import torch
    h, w_ = shape
    fp = wl.package_floorplan() if shape == (128, 128) else wl.toy_floorplan(h, w_, 8, 4, seed=h + w_)
    geo = wl.GEOMETRY["serving"] if shape == (128, 128) else wl.GEOMETRY["tiny"]
    prof = wl.load_profile("nominal", **geo, n_sub=9)
    a, b = hbf.Context(prof, fp), hbf.Context(prof, fp)
    b.set_thermal_path(True)
    dt = int(0.8 * a.euler_limit_ns() * 9)
    Ta = torch.empty(a.n_cells, dtype=torch.float32, device="cuda"); Tb = torch.empty_like(Ta)
    for k in range(30):
        ext = fp["ext_power_w"] * np.float32(1 + k % 4)
        hot_a = a.thermal_step(dt, ext, Ta)
        hot_b = b.thermal_step(dt, ext, Tb)
        assert torch.equal(Ta, Tb), k
        assert np.array_equal(hot_a, hot_b) and a.get_mode() == b.get_mode()
    assert np.array_equal(a.get_temps(), b.get_temps())
