"""The reduced-order thermal model on the device (hbf_rom_step) against the oracle's, and a model fitted by ERA from
the CUDA grid's own unit-step responses against the oracle's full grid (model against model, as the paper validates
its 224-state model)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import hbfo
from paper_2609_09800_b200 import era, workloads as wl


@pytest.fixture(scope="module")
def hbf():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_09800_b200 import build, hbf as mod
    build.build()
    return mod


@pytest.mark.parametrize("shape", [(224, 63, 11), (1, 1, 1), (37, 5, 70)])
def test_step_matches_the_oracle(hbf, shape):
    n, m, o = shape
    rng = np.random.default_rng(n)
    A = rng.normal(size=(n, n)); A *= 0.97 / max(np.abs(np.linalg.eigvals(A)).max(), 1e-9)
    B, C, D = rng.normal(size=(n, m)), rng.normal(size=(o, n)), rng.normal(size=(o, m))
    b, d = rng.normal(size=n) * 0.01, np.full(o, 35.0)
    g, r = hbf.Rom(A, B, C, D=D, b=b, d=d), hbfo.Rom(A, B, C, D=D, b=b, d=d)
    p = rng.uniform(0, 3, size=(400, m))
    Tg = np.vstack([g.step(p[:150]), g.step(p[150:])])      # the state carries over between calls
    Tr = r.step(p)
    scale = np.abs(Tr).max()
    assert np.abs(Tg - Tr).max() <= 1e-11 * scale            # double on both sides; only the summation order differs
    assert np.abs(g.state() - r.state()).max() <= 1e-11 * max(1.0, np.abs(r.state()).max())
    g.reset()
    assert not g.state().any()


def test_model_fitted_from_the_cuda_grid_tracks_the_oracle_grid(hbf):
    fp = wl.toy_floorplan(12, 24, 4, 2, seed=3)
    fp = dict(fp); fp["region_idle_w"] = np.zeros_like(fp["region_idle_w"])    # at rest the field is the ambient
    prof = wl.load_profile("nominal", channels=4, dies=2, planes=1, page_bytes=16384, stripe_bytes=16384, n_sub=8)
    prof.update(rtt_c=500.0, ltt_c=600.0, stt_c=700.0, shutdown_c=800.0)         # the controller stays Normal
    g = hbf.Context(prof, fp)
    dt = int(0.5 * g.euler_limit_ns()) * prof["n_sub"]
    region = np.asarray(fp["cell_region"])
    probes = [int(np.flatnonzero(region == k)[len(np.flatnonzero(region == k)) // 2]) for k in range(len(fp["region_kind"]))]
    K = 700
    steps = era.unit_step_responses(g, probes, K, dt)
    fit = era.era(era.markov_from_steps(steps), n_states=48, rows=300, cols=390)
    rom = hbf.Rom(fit["A"], fit["B"], fit["C"], D=fit["D"], d=np.full(len(probes), prof["ambient_c"]))
    # three input shapes, as in the paper's comparison: a step, a ramp, pulses; every region driven at once
    m = len(fp["region_kind"])
    n_run = 500
    k = np.arange(n_run)[:, None]
    amp = np.linspace(0.5, 2.0, m)[None, :]
    shapes = dict(step=np.ones((n_run, 1)) * amp, ramp=(k / n_run) * amp, pulses=((k // 40) % 2) * amp)
    worst = {}
    for name, p in shapes.items():
        o = hbfo.Oracle(prof, fp)
        full = np.empty((n_run, len(probes)))
        for i in range(n_run):
            _, T = o.thermal_step(dt, p[i].astype(np.float32), want_temps=True)
            full[i] = T[probes]
        rom.reset()
        red = rom.step(p.astype(np.float32).astype(np.float64))
        worst[name] = (np.abs(red - full).max(), full.max() - prof["ambient_c"])
    for name, (err, swing) in worst.items():
        assert err < 2e-3 * swing + 2e-3, (name, err, swing)   # within 0.2 % of the swing (the paper reports 0.07 % for its model)
    # steady state: the model's DC gain against the oracle grid driven to rest, one source
    o = hbfo.Oracle(prof, fp)
    p1 = np.zeros(m, np.float32); p1[2] = 1.0
    for _ in range(6000):
        hot, T = o.thermal_step(dt, p1, want_temps=True)
    assert np.abs(era.dc_gain(fit)[:, 2] - (T[probes] - prof["ambient_c"])).max() < 5e-3 * (T[probes].max() - prof["ambient_c"])


def test_context_steps_on_an_attached_model(hbf):
    """Coupled run with the thermal step on a reduced-order model: hot spots within 1e-9 K of the oracle's (double on
    both sides), the mode / service-fraction trace and every completion equal."""
    w = wl.prefix_kv(epochs=1, steps=1, batch=4, kv_tokens=256, layers=2)
    fp = wl.package_floorplan()
    prof = dict(w.profile); prof.update(rtt_c=36.0, ltt_c=36.6, stt_c=60.0, shutdown_c=90.0)   # thresholds the run crosses
    g, o = hbf.Context(prof, fp), hbfo.Oracle(prof, fp)
    for r in w.ranges:
        g.register_range(*r); o.register_range(*r)
    m = len(fp["region_kind"])
    rng = np.random.default_rng(5)
    n, no = 40, 9
    A = np.diag(rng.uniform(0.80, 0.97, n))
    B = rng.uniform(0.0, 0.02, size=(n, m)); C = rng.uniform(0.0, 0.05, size=(no, n)); D = rng.uniform(0.0, 0.002, size=(no, m))
    kinds = np.array([wl.KIND_HBF, wl.KIND_HBF, wl.KIND_HBF, wl.KIND_HBM, wl.KIND_HBM, wl.KIND_GPU, wl.KIND_GPU, wl.KIND_NONE, wl.KIND_HBF], np.int32)
    d = np.full(no, prof["ambient_c"])
    rg, ro = hbf.Rom(A, B, C, D=D, d=d, stream=g.stream), hbfo.Rom(A, B, C, D=D, d=d)
    dt = 1_000_000
    g.attach_rom(rg, kinds, dt)
    ext = fp["ext_power_w"]
    modes = set()
    for _, batch in wl.timed_batches(w, 14_000_000):
        rc_g, c_g, s_g, _, _ = g.submit_host(batch, check=False)
        rc_o, c_o, s_o, _, _ = o.submit(batch, check=False)
        assert rc_g == rc_o
        if rc_o == 0:
            assert np.array_equal(c_g, c_o) and np.array_equal(s_g, s_o)
        hot_g = g.thermal_step(dt, ext)
        hot_o = o.thermal_step_rom(ro, kinds, dt, ext)
        assert np.abs(hot_g.astype(np.float64) - hot_o).max() < 1e-4      # hot_c_out is float32
        assert np.abs(g.get_rom_temps()[kinds != wl.KIND_NONE].max() - hot_o.max()) < 1e-9
        assert g.get_mode() == o.mode()
        modes.add(o.mode()[0])
    assert len(modes) >= 2                                                 # the trace does leave Normal
    assert np.abs(rg.state() - ro.state()).max() < 1e-9
    with pytest.raises(hbf.HbfError):
        g.thermal_step(2 * dt, ext)                                        # the model was fitted for one step length
    g.attach_rom(None)
    g.thermal_step(dt, ext)                                                # the grid again
