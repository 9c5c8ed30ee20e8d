"""The allocation-free Euler entry point against hbf_thermal_step, through the C ABI.

Some callers of this library may not allocate device memory (a serving loop that cannot take the
device-wide stall cudaMalloc can cause; a plug-in confined to buffers its host hands it).  For them
``hbf_euler_substeps_static`` keeps its second field buffer in an array built into the library.  This
test drives it twice in a row on caller-owned buffers and compares the field with what the regular,
context-based ``hbf_thermal_step`` produces for the same floorplan and power, and with the float64 CPU
oracle's thermal step, within the 1e-3 K tolerance the thermal parity tests use; the free device
memory the CUDA runtime reports must not move across the call.  The file sorts last so that a run which stops at the first
failure has already run everything else.
"""
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


def cell_power(fp, ext):
    """Watts per cell exactly as the library's power map forms them with no die energy pending."""
    region = np.asarray(fp["cell_region"])
    pr = np.asarray(fp["region_idle_w"], np.float32).astype(np.float64) + np.asarray(ext, np.float32).astype(np.float64)
    cnt = np.bincount(region[region >= 0], minlength=pr.shape[0]).astype(np.float64)
    inv = np.where(cnt > 0, 1.0 / np.maximum(cnt, 1), 0.0).astype(np.float32).astype(np.float64)
    return np.where(region >= 0, pr[np.maximum(region, 0)] * inv[np.maximum(region, 0)], 0.0).astype(np.float32)


@pytest.mark.parametrize("plan", ["package", "toy"])
def test_static_entry_matches_thermal_step_on_two_calls_in_a_row(hbf, plan):
    import torch
    if plan == "package":
        fp, prof = wl.package_floorplan(), wl.load_profile("nominal", **wl.GEOMETRY["serving"])
    else:
        fp, prof = wl.toy_floorplan(37, 53, 8, 4, seed=4), wl.load_profile("nominal", **wl.GEOMETRY["tiny"], n_sub=7)
    ctx = hbf.Context(prof, fp)
    n_sub = prof["n_sub"]
    dt_ns = int(0.8 * ctx.euler_limit_ns() * n_sub)
    dt_sub = np.float32(dt_ns * 1e-9 / n_sub)               # the float the library itself derives
    dev = lambda a, dt=torch.float32: torch.from_numpy(np.ascontiguousarray(a)).to("cuda", dt)
    C_, Gx, Gy, Gs = (dev(fp[k]) for k in ("cell_C", "cell_Gx", "cell_Gy", "cell_Gsink"))
    n_cells = fp["grid_h"] * fp["grid_w"]
    theta = torch.zeros(n_cells, dtype=torch.float32, device="cuda")
    comp = torch.zeros(n_cells, dtype=torch.float32, device="cuda")
    d_T = torch.empty(n_cells, dtype=torch.float32, device="cuda")
    orc = hbfo.Oracle(prof, fp)                             # float64, cell by cell: the independent reference
    # warm-up on scratch buffers of its own: module load and the look-up of the built-in array's address happen here
    w_theta, w_comp = torch.zeros_like(theta), torch.zeros_like(comp)
    P0 = dev(cell_power(fp, fp["ext_power_w"]))
    assert hbf.euler_substeps_static(C_, Gx, Gy, Gs, P0, w_theta, w_comp, fp["grid_h"], fp["grid_w"], 1, float(dt_sub)) == hbf.OK
    torch.cuda.synchronize()
    for call, scale in enumerate((1.0, 2.5)):               # two calls in a row, the second with other power
        ext = fp["ext_power_w"] * np.float32(scale)
        P = dev(cell_power(fp, ext))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]          # what cudaMemGetInfo reports: sees any cudaMalloc, torch's or not
        rc = hbf.euler_substeps_static(C_, Gx, Gy, Gs, P, theta, comp, fp["grid_h"], fp["grid_w"], n_sub, float(dt_sub))
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        assert rc == hbf.OK
        ctx.thermal_step(dt_ns, ext, d_T)
        _, t_o = orc.thermal_step(dt_ns, ext, want_temps=True)
        torch.cuda.synchronize()
        got = theta.cpu().numpy().astype(np.float64) + prof["ambient_c"]
        want = d_T.cpu().numpy().astype(np.float64)
        assert np.abs(got - want).max() < TOL_K, (plan, call)
        assert np.abs(got - t_o).max() < TOL_K, (plan, call, "oracle")
        assert want.max() > prof["ambient_c"] + 1e-4        # the step did something
    # odd substep counts end in the built-in buffer and are copied back
    theta2 = torch.zeros(n_cells, dtype=torch.float32, device="cuda"); comp2 = torch.zeros_like(theta2)
    theta3 = torch.zeros(n_cells, dtype=torch.float32, device="cuda"); comp3 = torch.zeros_like(theta3)
    assert hbf.euler_substeps_static(C_, Gx, Gy, Gs, P, theta2, comp2, fp["grid_h"], fp["grid_w"], 3, float(dt_sub)) == hbf.OK
    for _ in range(3):
        assert hbf.euler_substeps_static(C_, Gx, Gy, Gs, P, theta3, comp3, fp["grid_h"], fp["grid_w"], 1, float(dt_sub)) == hbf.OK
    assert torch.equal(theta2, theta3) and torch.equal(comp2, comp3)


def test_static_entry_rejects_oversized_grids_and_bad_arguments(hbf):
    import torch
    t = torch.zeros(16, dtype=torch.float32, device="cuda")
    assert hbf.euler_substeps_static(t, t, t, t, t, t, t, 257, 256, 1, 1e-5) == hbf.E_WORKSPACE
    assert hbf.STATIC_MAX_CELLS == 256 * 256
    assert hbf.euler_substeps_static(t, t, t, t, t, t, t, 4, 4, 0, 1e-5) == hbf.E_INVAL
    assert hbf.euler_substeps_static(t, t, t, t, t, None, t, 4, 4, 1, 1e-5) == hbf.E_INVAL
    assert hbf.euler_substeps_static(t, t, t, t, t, t, t, 4, 4, 1, 0.0) == hbf.E_INVAL
