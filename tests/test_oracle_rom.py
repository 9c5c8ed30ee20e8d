"""Pins of the oracle's reduced-order thermal model step (Eq. 2): closed forms and textbook special cases."""
import numpy as np
import pytest

from oracle import hbfo


def test_scalar_system_closed_form():
    a, bb, c, dd, b0, d0 = 0.9, 0.5, 2.0, 0.25, 0.1, 30.0
    rom = hbfo.Rom([[a]], [[bb]], [[c]], D=[[dd]], b=[b0], d=[d0])
    T = rom.step(np.ones((50, 1)))
    # x_k = (bb + b0) (1 - a^k) / (1 - a); T_k = c x_k + dd + d0 (x_k is the state before step k's update)
    k = np.arange(50)
    want = c * (bb + b0) * (1 - a ** k) / (1 - a) + dd + d0
    assert np.allclose(T[:, 0], want, rtol=1e-13, atol=0)
    assert T[0, 0] == dd + d0                              # at the first sample only the feedthrough and the offset show


def test_impulse_response_gives_the_markov_parameters():
    rng = np.random.default_rng(0)
    n, m, o = 7, 3, 4
    A = rng.normal(size=(n, n)); A *= 0.8 / np.abs(np.linalg.eigvals(A)).max()
    B, Cm, D = rng.normal(size=(n, m)), rng.normal(size=(o, n)), rng.normal(size=(o, m))
    for j in range(m):
        rom = hbfo.Rom(A, B, Cm, D=D)
        p = np.zeros((12, m)); p[0, j] = 1.0
        T = rom.step(p)
        assert np.allclose(T[0], D[:, j], atol=1e-15)
        Ak = np.eye(n)
        for k in range(1, 12):                               # h_k = C A^(k-1) B
            assert np.allclose(T[k], (Cm @ Ak @ B)[:, j], rtol=1e-12, atol=1e-14)
            Ak = Ak @ A


def test_steady_state_is_the_dc_gain_and_steps_chain():
    rng = np.random.default_rng(1)
    n, m, o = 5, 2, 3
    A = np.diag(rng.uniform(0.2, 0.9, n)); B, Cm = rng.normal(size=(n, m)), rng.normal(size=(o, n))
    d = np.full(o, 35.0)
    rom = hbfo.Rom(A, B, Cm, d=d)
    p = np.tile([[1.5, -0.5]], (600, 1))
    T = rom.step(p)
    gain = Cm @ np.linalg.solve(np.eye(n) - A, B)            # R_ij = dT_i / P_j, K/W
    assert np.allclose(T[-1], d + gain @ p[0], rtol=1e-10)
    rom.reset()
    T2 = np.vstack([rom.step(p[:250]), rom.step(p[250:])])  # the state carries over between calls
    assert np.array_equal(T, T2)
    rom.reset()
    assert not rom.state().any()


def test_thermal_step_on_the_model_uses_the_same_power_vector(golden_dir):
    """A model that is pure feedthrough, T = ambient + R p, shows the power vector itself: the paper's read power,
    384e9 B/s x 84 pJ/B + 5 W idle = 37.256 W, and the controller acting on the resulting temperature."""
    import json, os
    from paper_2609_09800_b200 import workloads as wl
    with open(os.path.join(golden_dir, "paper_values.json")) as f:
        pv = json.load(f)["hbf_read_power"]
    prof = wl.load_profile("nominal", channels=16, dies=8, planes=1, page_bytes=16384, stripe_bytes=65536, n_sub=1)
    prof.update(rtt_c=60.0, ltt_c=100.0, stt_c=120.0, shutdown_c=150.0)
    fp = dict(grid_h=1, grid_w=1, cell_C=[1000.0], cell_Gx=[0.0], cell_Gy=[0.0], cell_Gsink=[1.0], cell_region=[0],
              die_region=[0] * 128, region_kind=[wl.KIND_HBF], region_idle_w=[pv["idle_w"]])
    o = hbfo.Oracle(prof, fp)
    o.register_range(wl.RANGE_BASE, 1 << 40)
    n = int(pv["bytes_per_s"]) // 65536
    acc = np.zeros(n, hbfo.ACCESS_DTYPE)
    acc["addr"] = wl.RANGE_BASE + np.arange(n, dtype=np.uint64) * np.uint64(65536)
    acc["bytes"] = 65536
    o.submit(acc)
    rom = hbfo.Rom(np.zeros((1, 1)), np.zeros((1, 1)), np.zeros((1, 1)), D=[[2.0]], d=[prof["ambient_c"]])   # 2 K/W
    hot = o.thermal_step_rom(rom, [wl.KIND_HBF], 1_000_000_000)
    assert hot[0] - prof["ambient_c"] == pytest.approx(2.0 * pv["power_w"], abs=1e-9)
    assert not o.pending_energy().any()
    assert o.mode()[0] == hbfo.MODE_LIGHT              # 35 + 74.5 = 109.5 C: above the light threshold, below severe
    hot = o.thermal_step_rom(rom, [wl.KIND_HBF], 1_000_000_000)    # no traffic any more: idle power only, 35 + 10 C
    assert hot[0] - prof["ambient_c"] == pytest.approx(2.0 * pv["idle_w"], abs=1e-12)
    assert o.mode()[0] == hbfo.MODE_NORMAL             # back below the release threshold
