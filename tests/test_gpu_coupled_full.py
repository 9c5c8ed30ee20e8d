"""The long coupled run at its full length: 10 s of simulated time in 10,000 batches of 1 ms, each followed by a thermal
step on the 128x128 package grid, on the nominal and on the aggressive timing profile.

Every batch is served by the library (through the C ABI) and by the CPU oracle; compared are every completion, stall
and per-die statistic, the batch summaries, the queue state, the mode / service-fraction trace after every step, the
three hotspot temperatures after every step and the whole field every 100 steps (1e-3 K).  Where the two sides take a
different throttle decision while the oracle's hotspot lies within 2e-3 K of a threshold (float32 against float64 at a
threshold quantised to mK), the oracle is moved to the library's mode and the run goes on; any other divergence fails.
The stream is the shared-prefix KV + weights stream, repeated back to back until the horizon (at 50 % load that is
about 6e7 accesses on the nominal profile and five times as many on the aggressive one)."""
import time

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import hbfo
from paper_2609_09800_b200 import workloads as wl

TOL_K = 1e-3
HORIZON_NS, WINDOW_NS = 10_000_000_000, 1_000_000


@pytest.fixture(scope="module")
def hbf():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_09800_b200 import build, hbf as mod
    build.build()
    return mod


def near_threshold(prof, t_hot_c, tol=2e-3):
    return any(abs(t_hot_c - prof[k]) <= tol for k in ("rtt_c", "ltt_c", "stt_c", "shutdown_c"))


@pytest.mark.parametrize("profile", ["nominal", "aggressive"])
def test_ten_seconds_in_one_millisecond_batches(hbf, profile):
    import torch
    w = wl.prefix_kv(profile=profile)
    fp = wl.package_floorplan()
    g, o = hbf.Context(w.profile, fp), hbfo.Oracle(w.profile, fp)
    for r in w.ranges:
        g.register_range(*r); o.register_range(*r)
    ext = fp["ext_power_w"]
    d_T = torch.empty(g.n_cells, dtype=torch.float32, device="cuda")
    trace, ties, refused, served = [], 0, 0, 0
    t_gpu = t_cpu = 0.0
    steps = 0
    for k, acc in wl.timed_batches(w, HORIZON_NS, WINDOW_NS):
        t0 = time.perf_counter()
        rc_o, c_o, s_o, st_o, ds_o = o.submit(acc, check=False)
        t1 = time.perf_counter()
        rc_g, c_g, s_g, st_g, ds_g = g.submit_host(acc, check=False)
        t2 = time.perf_counter()
        assert rc_g == rc_o, (k, rc_g, rc_o)
        assert g.last_result() == o.last_result(), k
        if rc_o == 0:
            bad = np.flatnonzero(c_g != c_o)
            assert bad.size == 0, "step %d: first mismatch at %d: gpu %d oracle %d" % (k, bad[0], c_g[bad[0]], c_o[bad[0]])
            assert np.array_equal(s_g, s_o) and np.array_equal(st_g, st_o)
            for f in hbfo.DIE_STATS_DTYPE.names:
                assert np.array_equal(ds_g[f], ds_o[f]), (k, f)
            served += acc.shape[0]
        else:
            assert rc_o in (hbfo.E_THROTTLED, hbfo.E_LINK_SHUTDOWN), (k, rc_o)
            refused += 1
        want_field = k % 100 == 99
        t3 = time.perf_counter()
        hot_g = g.thermal_step(WINDOW_NS, ext, d_T if want_field else None)
        t4 = time.perf_counter()
        hot_o, T_o = o.thermal_step(WINDOW_NS, ext, want_temps=want_field)
        t5 = time.perf_counter()
        t_cpu += (t1 - t0) + (t5 - t4); t_gpu += (t2 - t1) + (t4 - t3)
        assert np.abs(hot_g.astype(np.float64) - hot_o).max() < TOL_K, (k, hot_g, hot_o)
        if want_field:
            assert np.abs(d_T.cpu().numpy().astype(np.float64) - T_o).max() < TOL_K, k
            assert np.array_equal(g.get_busy_until(), o.busy_until()), k
            assert np.array_equal(g.get_pending_energy(), o.pending_energy()), k
        mg, mo = g.get_mode(), o.mode()
        if mg != mo:
            assert near_threshold(w.profile, float(hot_o[0])), (k, mg, mo, hot_o)
            o.force_mode(*mg); ties += 1                     # threshold tie: follow the library and go on
        trace.append(mg[0])
        steps += 1
    assert steps == HORIZON_NS // WINDOW_NS
    assert np.array_equal(g.get_busy_until(), o.busy_until())
    modes = sorted(set(trace))
    print("\n%s: %d steps, %d accesses served, %d batches refused by the controller, modes seen %s, %d threshold ties; "
          "hottest HBF cell at the end %.3f C; wall time library side %.1f s (host copies included), oracle side %.1f s"
          % (profile, steps, served, refused, modes, ties, float(hot_o[0]), t_gpu, t_cpu))
    assert served > 5e7 * (1 if profile == "nominal" else 1) or refused > 0
    assert hot_o[0] > w.profile["ambient_c"] + 20.0           # the package did heat up
    if profile == "nominal":
        assert hbf.MODE_LIGHT in modes and refused == 0       # crosses the light threshold, never the severe one
