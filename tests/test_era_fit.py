"""The ERA fit (numpy, offline) recovers a known system from its step responses; no GPU needed."""
import numpy as np

from oracle import hbfo
from paper_2609_09800_b200 import era


def known_system(seed, n=6, m=3, o=4):
    rng = np.random.default_rng(seed)
    A = rng.normal(size=(n, n)); A *= 0.9 / np.abs(np.linalg.eigvals(A)).max()
    return A, rng.normal(size=(n, m)), rng.normal(size=(o, n)), rng.normal(size=(o, m))


def step_responses(A, B, C, D, K):
    """unit step on each input, recorded with the oracle's reduced-model step"""
    m, o = B.shape[1], C.shape[0]
    out = np.empty((K, o, m))
    for j in range(m):
        p = np.zeros((K, m)); p[:, j] = 1.0
        out[:, :, j] = hbfo.Rom(A, B, C, D=D).step(p)
    return out


def test_fit_reproduces_the_markov_parameters_and_the_dc_gain():
    A, B, C, D = known_system(3)
    steps = step_responses(A, B, C, D, 80)
    h = era.markov_from_steps(steps)
    assert np.allclose(h[0], D) and np.allclose(h[1], C @ B) and np.allclose(h[2], C @ A @ B)
    fit = era.era(h, n_states=6)
    assert fit["A"].shape == (6, 6)
    assert np.allclose(np.sort_complex(np.linalg.eigvals(fit["A"])), np.sort_complex(np.linalg.eigvals(A)), atol=1e-8)
    Ak = np.eye(6)
    for k in range(1, 40):                                  # the realisation differs by a similarity transform; its responses do not
        assert np.allclose(fit["C"] @ np.linalg.matrix_power(fit["A"], k - 1) @ fit["B"], C @ Ak @ B, atol=1e-8)
        Ak = Ak @ A
    assert np.allclose(era.dc_gain(fit), D + C @ np.linalg.solve(np.eye(6) - A, B), atol=1e-7)
    # a fitted model driven by an arbitrary input follows the original one
    rng = np.random.default_rng(0)
    p = rng.uniform(0, 2, size=(200, 3))
    want = hbfo.Rom(A, B, C, D=D).step(p)
    got = hbfo.Rom(fit["A"], fit["B"], fit["C"], D=fit["D"]).step(p)
    assert np.abs(got - want).max() < 1e-7


def test_truncation_keeps_the_dominant_modes():
    A = np.diag([0.95, 0.9, 0.5, 0.01]); B = np.ones((4, 1)); C = np.array([[1.0, 1.0, 1.0, 1e-6]])
    h = era.markov_from_steps(step_responses(A, B, C, np.zeros((1, 1)), 120))
    fit = era.era(h, n_states=3)
    assert np.allclose(np.sort(np.linalg.eigvals(fit["A"]).real), [0.5, 0.9, 0.95], atol=1e-5)
