"""SHA-256 fingerprints of the seeded synthetic streams, so that a change of numpy (or of a generator) that reshuffles a
stream cannot go unseen: every result quoted for a stream is a result for exactly these bytes.

``python -m paper_2609_09800_b200.config.fingerprint_streams`` recomputes all of them and rewrites ``streams.json`` beside
this file; ``--cheap`` leaves the two largest out (the tests do the same on the CPU machine and check those two on the GPU machine).
"""
from __future__ import annotations

import hashlib
import json
import os
import sys

import numpy as np

from paper_2609_09800_b200 import workloads as wl

HERE = os.path.dirname(os.path.abspath(__file__))
FILE = os.path.join(HERE, "streams.json")

# name -> (maker, cheap enough for the CPU test suite)
STREAMS = {
    "tiny_uniform(65536, seed 0)": (lambda: wl.tiny_uniform().acc, True),
    "decode_weights(48 tokens, seed 0)": (lambda: wl.decode_weights(48).acc, True),
    "decode_weights(256 tokens, seed 0)": (lambda: wl.decode_weights(256).acc, False),
    "prefix_kv(seed 0)": (lambda: wl.prefix_kv().acc, False),
    "capacity_mode(first 8,000,000 of any length, seed 0)": (lambda: wl.capacity_mode(n=8_000_000).acc, True),
    "capacity_mode(200,000,000, seed 0)": (lambda: wl.capacity_mode(n=200_000_000).acc, False),
    "mixed_status(10000, seed 0, faults)": (lambda: wl.mixed_status(10_000, seed=0, faults=True).acc, True),
    "package_floorplan(): C, Gx, Gy, Gsink, region, die_region": (
        lambda: np.concatenate([np.asarray(wl.package_floorplan()[k]).astype(np.float64).ravel()
                                for k in ("cell_C", "cell_Gx", "cell_Gy", "cell_Gsink", "cell_region", "die_region")]), True),
}


def sha256_of(arr: np.ndarray) -> str:
    a = np.ascontiguousarray(arr)
    h = hashlib.sha256()
    view = memoryview(a).cast("B")
    step = 1 << 28
    for lo in range(0, len(view), step):
        h.update(view[lo:lo + step])
    return h.hexdigest()


def compute(cheap_only: bool = False) -> dict:
    return {name: sha256_of(make()) for name, (make, cheap) in STREAMS.items() if cheap or not cheap_only}


def recorded() -> dict:
    with open(FILE) as f:
        return json.load(f)


if __name__ == "__main__":
    cheap = "--cheap" in sys.argv
    rec = recorded() if os.path.exists(FILE) else {"sha256": {}}
    rec["numpy"] = np.__version__
    rec["generator"] = "numpy.random.Generator(PCG64([seed, stream]))"
    rec["sha256"].update(compute(cheap))
    with open(FILE, "w") as f:
        json.dump(rec, f, indent=1, sort_keys=True)
        f.write("\n")
    print(json.dumps(rec, indent=1, sort_keys=True))
