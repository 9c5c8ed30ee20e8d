"""Offline fit of the reduced-order thermal model (Eq. 2) by the Eigensystem Realization Algorithm.

The paper's procedure: every heat source receives a 1 W unit step on the full package operator, and ERA fits a
discrete state-space model to the recorded response.  Here the full operator is this library's own RC grid
(`hbf_thermal_step`); `unit_step_responses` records it, `era` fits `(A, B, C, D)`, and the result is stepped at run
time by `hbf_rom_step`.  Plain numpy, run once per floorplan; not on the per-step path."""
from __future__ import annotations

import numpy as np


def markov_from_steps(steps: np.ndarray) -> np.ndarray:
    """steps [K][outputs][inputs]: response at sample k to a unit step applied from sample 0 on (rise above the
    operating point).  Returns the impulse response h [K][outputs][inputs] (h_0 = D, h_k = C A^(k-1) B)."""
    steps = np.asarray(steps, np.float64)
    h = steps.copy()
    h[1:] -= steps[:-1]
    return h


def era(h: np.ndarray, n_states: int, rows: int | None = None, cols: int | None = None):
    """Eigensystem Realization Algorithm on the impulse response h [K][outputs][inputs].

    Block Hankel matrices H0[i][j] = h[i+j+1], H1[i][j] = h[i+j+2]; H0 = U S V^T truncated to n_states;
    A = S^-1/2 U^T H1 V S^-1/2, B = first block column of S^1/2 V^T, C = first block row of U S^1/2, D = h[0].
    Returns dict(A, B, C, D, singular_values)."""
    h = np.asarray(h, np.float64)
    K, p, m = h.shape
    rows = rows if rows is not None else (K - 2) // 2
    cols = cols if cols is not None else K - 2 - rows
    assert rows >= 1 and cols >= 1 and rows + cols + 1 <= K, "impulse response too short for the Hankel matrices"
    H0 = np.empty((rows * p, cols * m)); H1 = np.empty_like(H0)
    for i in range(rows):
        for j in range(cols):
            H0[i * p:(i + 1) * p, j * m:(j + 1) * m] = h[i + j + 1]
            H1[i * p:(i + 1) * p, j * m:(j + 1) * m] = h[i + j + 2]
    U, s, Vt = np.linalg.svd(H0, full_matrices=False)
    n = int(min(n_states, (s > s[0] * 1e-14).sum()))
    U, sv, Vt = U[:, :n], s[:n], Vt[:n]
    sq = np.sqrt(sv)
    A = (U / sq).T @ H1 @ (Vt.T / sq)
    B = (sq[:, None] * Vt)[:, :m]
    C = (U * sq)[:p]
    return dict(A=A, B=B, C=C, D=h[0].copy(), singular_values=s)


def dc_gain(rom: dict) -> np.ndarray:
    """Steady-state temperature change per watt, R_ij = dT_i / P_j (K/W), of a fitted model."""
    n = rom["A"].shape[0]
    return rom["D"] + rom["C"] @ np.linalg.solve(np.eye(n) - rom["A"], rom["B"])


def unit_step_responses(ctx, probes, n_steps: int, dt_ns: int, inputs=None) -> np.ndarray:
    """Records the full grid's response at the probe cells to a 1 W step on each region in turn, through
    `hbf_thermal_step` of the given context (its per-region idle powers should be zero, so that the field at rest is
    the ambient).  Returns steps [n_steps][len(probes)][n_inputs]: sample k is the rise above ambient after k + 1
    steps, i.e. the output of the step during which input sample k was applied."""
    import torch
    n_regions = ctx.n_regions
    inputs = list(range(n_regions)) if inputs is None else list(inputs)
    probes_t = torch.as_tensor(np.asarray(probes, np.int64), device="cuda")
    d_temps = torch.empty(ctx.n_cells, dtype=torch.float32, device="cuda")
    out = np.empty((n_steps, len(probes), len(inputs)), np.float64)
    ambient = float(ctx.ambient_c)
    rec = torch.empty((n_steps, len(probes)), dtype=torch.float32, device="cuda")
    for col, j in enumerate(inputs):
        ctx.reset()
        ext = np.zeros(n_regions, np.float32); ext[j] = 1.0
        for k in range(n_steps):
            ctx.thermal_step(dt_ns, ext, d_temps, want_hot=False)
            rec[k] = d_temps[probes_t]
        out[:, :, col] = rec.cpu().numpy().astype(np.float64) - ambient
    ctx.reset()
    return out
