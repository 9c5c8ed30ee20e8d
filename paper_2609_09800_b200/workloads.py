"""Seeded synthetic inputs: timing profiles, HBF geometries, access streams and the package floorplan.

This module only *makes inputs*.  It holds none of the service model's arithmetic and is the one
module that both the CUDA library's callers and the CPU oracle's callers use.  Every stream is a
numpy structured array of 24-byte access records ``(addr u64, issue_ns i64, bytes u32, flags u32)``
drawn from ``numpy.random.Generator(PCG64(seed))``.

The streams stand in for the paper's workloads (Qwen3-30B-A3B served by an inference framework, and
a captured expert-routing trace), none of which are available offline: only the tensor *shapes* of
that model are used (48 layers, hidden 2048, 128 experts of intermediate 768, top-8, 4 KV heads of
128, bf16), which reproduce the paper's 54.000 GiB expert set (EQ3).
"""
from __future__ import annotations

import json
import os
from dataclasses import dataclass, field

import numpy as np

ACCESS_DTYPE = np.dtype([("addr", "<u8"), ("issue_ns", "<i8"), ("bytes", "<u4"), ("flags", "<u4")])
assert ACCESS_DTYPE.itemsize == 24

RANGE_BASE = 0x7000_0000_0000
KIB, MIB, GIB = 1 << 10, 1 << 20, 1 << 30
PERM_R, PERM_P = 1, 2
KIND_NONE, KIND_GPU, KIND_HBM, KIND_HBF = 0, 1, 2, 3

_CFG_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "config")


def load_profile(name: str = "nominal", **geometry) -> dict:
    """Timing/energy/thermal scalars of a committed profile merged with a geometry."""
    with open(os.path.join(_CFG_DIR, name + ".json")) as f:
        prof = {k: v for k, v in json.load(f).items() if not k.startswith("_")}
    prof.update(geometry)
    return prof


GEOMETRY = {
    "tiny":     dict(channels=8,  dies=4, planes=2, page_bytes=16 * KIB, stripe_bytes=16 * KIB),
    "serving":  dict(channels=32, dies=8, planes=4, page_bytes=16 * KIB, stripe_bytes=64 * KIB),
    "capacity": dict(channels=64, dies=8, planes=4, page_bytes=16 * KIB, stripe_bytes=64 * KIB),
}

# ---- Qwen3-30B-A3B-shaped weight image (layer-major) ------------------------------------------
N_LAYERS, HIDDEN, N_EXPERTS, EXPERT_INTER, TOP_K = 48, 2048, 128, 768, 8
TILE = 64 * KIB
ATTN_BYTES = 2 * (HIDDEN * 4096 + 2 * HIDDEN * 512 + 4096 * HIDDEN)        # q, k, v, o in bf16
EXPERT_BYTES = 2 * 3 * HIDDEN * EXPERT_INTER                               # gate, up, down in bf16
LAYER_BYTES = ATTN_BYTES + N_EXPERTS * EXPERT_BYTES
WEIGHT_BYTES = N_LAYERS * LAYER_BYTES
ATTN_TILES, EXPERT_TILES = ATTN_BYTES // TILE, EXPERT_BYTES // TILE
assert (ATTN_TILES, EXPERT_TILES) == (576, 144)
assert N_LAYERS * N_EXPERTS * EXPERT_BYTES == 54 * GIB                     # the paper's expert set
KV_OFFSET = 56 * GIB
KV_TOKENS, KV_BYTES_PER_TOKEN_LAYER = 8192, 2 * 4 * 128 * 2               # K+V, 4 heads x 128, bf16
KV_LAYER_BYTES = KV_TOKENS * KV_BYTES_PER_TOKEN_LAYER                     # 16 MiB
KV_BYTES = N_LAYERS * KV_LAYER_BYTES                                      # 768 MiB
SERVING_RANGE = 57 * GIB


@dataclass
class Workload:
    """A stream plus everything needed to set a context up for it."""
    name: str
    profile: dict
    ranges: list                      # [(base, length, perms, kind, stream_tag, media_offset)]
    acc: np.ndarray
    meta: dict = field(default_factory=dict)

    @property
    def n(self) -> int:
        return int(self.acc.shape[0])


def _poisson_issue(rng: np.random.Generator, n: int, mean_gap_ns: float, t0: float = 0.0):
    """floor(cumsum(Exp(mean))) as int64 ns, plus the carry for a following chunk."""
    t = t0 + np.cumsum(rng.exponential(mean_gap_ns, n))
    return np.floor(t).astype(np.int64), (float(t[-1]) if n else t0)


def _records(addr, issue, nbytes, flags) -> np.ndarray:
    out = np.empty(len(addr), ACCESS_DTYPE)
    out["addr"], out["issue_ns"], out["bytes"], out["flags"] = addr, issue, nbytes, flags
    return out


# ---- config 1: tiny uniform read stream ---------------------------------------------------------

def tiny_uniform(n: int = 65536, seed: int = 0, rho: float = 0.5, profile: str = "nominal") -> Workload:
    prof = load_profile(profile, **GEOMETRY["tiny"])
    rng = np.random.Generator(np.random.PCG64([seed, 1]))
    R = 8 * 4 * 2
    mean_gap = prof["t_read_ns"] / (rho * R)                  # one-page reads on R queues at load rho
    addr = RANGE_BASE + rng.integers(0, GIB // (4 * KIB), n, dtype=np.uint64) * np.uint64(4 * KIB)
    issue, _ = _poisson_issue(rng, n, mean_gap)
    acc = _records(addr, issue, 4 * KIB, 0)
    return Workload("tiny_uniform", prof, [(RANGE_BASE, GIB, PERM_R | PERM_P, 0, 0, 0)], acc,
                    dict(rho=rho, mean_gap_ns=mean_gap, queues=R))


# ---- config 2: decode weight streaming -----------------------------------------------------------

def _expert_perms(rng):
    return np.stack([rng.permutation(N_EXPERTS) for _ in range(N_LAYERS)])          # [layer, rank] -> expert


def _route_topk(rng, perms, n_tokens):
    """Top-8 of 128 without replacement, weights rank^-1.1 (Gumbel top-k), per token and layer."""
    logw = -1.1 * np.log(np.arange(1, N_EXPERTS + 1, dtype=np.float64))
    g = rng.gumbel(size=(n_tokens, N_LAYERS, N_EXPERTS))
    ranks = np.argsort(-(logw + g), axis=-1)[..., :TOP_K]                            # ranks drawn
    return np.take_along_axis(np.broadcast_to(perms, (n_tokens,) + perms.shape), ranks, axis=-1)


def decode_weights(tokens: int = 256, seed: int = 0, rho: float = 0.5, profile: str = "nominal") -> Workload:
    prof = load_profile(profile, **GEOMETRY["serving"])
    rng = np.random.Generator(np.random.PCG64([seed, 2]))
    perms = _expert_perms(rng)
    experts = _route_topk(rng, perms, tokens)                                        # [tok, layer, 8]
    layer_off = (np.arange(N_LAYERS, dtype=np.int64) * LAYER_BYTES)[None, :, None]
    attn = layer_off + (np.arange(ATTN_TILES, dtype=np.int64) * TILE)[None, None, :]             # [1, L, 576]
    attn = np.broadcast_to(attn, (tokens, N_LAYERS, ATTN_TILES))
    ex = (layer_off[..., None] + ATTN_BYTES + experts[..., None].astype(np.int64) * EXPERT_BYTES
          + (np.arange(EXPERT_TILES, dtype=np.int64) * TILE)[None, None, None, :])               # [tok, L, 8, 144]
    off = np.concatenate([attn, ex.reshape(tokens, N_LAYERS, TOP_K * EXPERT_TILES)], axis=2).reshape(-1)
    n = off.shape[0]
    R = 32 * 8 * 4
    mean_gap = 4 * prof["t_read_ns"] / (rho * R)
    issue, _ = _poisson_issue(rng, n, mean_gap)
    acc = _records(RANGE_BASE + off.astype(np.uint64), issue, TILE, 0)
    return Workload("decode_weights", prof, [(RANGE_BASE, SERVING_RANGE, PERM_R | PERM_P, 0, 0, 0)], acc,
                    dict(rho=rho, mean_gap_ns=mean_gap, queues=R, tokens=tokens))


# ---- config 3: shared-prefix KV cache plus weights ---------------------------------------------------

def prefix_kv(epochs: int = 3, steps: int = 6, batch: int = 64, seed: int = 0, rho: float = 0.5,
              profile: str = "nominal", kv_tokens: int = KV_TOKENS, layers: int = N_LAYERS) -> Workload:
    """Per epoch: program the shared prefix KV as 4 KiB programs in address order, then ``steps``
    decode steps at ``batch`` requests: per layer the attention tiles once, the union of the
    requests' routed experts once each, and every request reading that layer's prefix KV tiles."""
    prof = load_profile(profile, **GEOMETRY["serving"])
    rng = np.random.Generator(np.random.PCG64([seed, 3]))
    perms = _expert_perms(rng)
    kv_layer_bytes = kv_tokens * KV_BYTES_PER_TOKEN_LAYER
    kv_tiles = max(1, kv_layer_bytes // TILE)
    offs, sizes, flags = [], [], []
    for _ in range(epochs):
        n_prog = layers * kv_layer_bytes // (4 * KIB)
        offs.append(KV_OFFSET + np.arange(n_prog, dtype=np.int64) * (4 * KIB))
        sizes.append(np.full(n_prog, 4 * KIB, np.uint32)); flags.append(np.ones(n_prog, np.uint32))
        for _ in range(steps):
            experts = _route_topk(rng, perms, batch)                                   # [batch, L, 8]
            for l in range(layers):
                uni = np.unique(experts[:, l, :])
                base = l * LAYER_BYTES
                a = base + np.arange(ATTN_TILES, dtype=np.int64) * TILE
                e = (base + ATTN_BYTES + uni.astype(np.int64)[:, None] * EXPERT_BYTES
                     + np.arange(EXPERT_TILES, dtype=np.int64)[None, :] * TILE).reshape(-1)
                kv = np.tile(KV_OFFSET + l * kv_layer_bytes + np.arange(kv_tiles, dtype=np.int64) * TILE, batch)
                o = np.concatenate([a, e, kv])
                offs.append(o); sizes.append(np.full(o.shape[0], TILE, np.uint32))
                flags.append(np.zeros(o.shape[0], np.uint32))
    off = np.concatenate(offs); nbytes = np.concatenate(sizes); fl = np.concatenate(flags)
    n = off.shape[0]
    R = 32 * 8 * 4
    frac_prog = float(fl.mean())
    mean_service = frac_prog * prof["t_prog_ns"] + (1.0 - frac_prog) * 4 * prof["t_read_ns"]
    mean_gap = mean_service / (rho * R)
    issue, _ = _poisson_issue(rng, n, mean_gap)
    acc = _records(RANGE_BASE + off.astype(np.uint64), issue, nbytes, fl)
    return Workload("prefix_kv", prof, [(RANGE_BASE, SERVING_RANGE, PERM_R | PERM_P, 0, 0, 0)], acc,
                    dict(rho=rho, mean_gap_ns=mean_gap, queues=R, frac_program=frac_prog))


# ---- config 4: capacity mode -------------------------------------------------------------------------

CAPACITY_REPLICAS, CAPACITY_SLOT = 16, 96 * GIB
CAPACITY_RANGE = CAPACITY_REPLICAS * CAPACITY_SLOT                       # 1.5 TiB


def _capacity_chunk(seed: int, k: int, m: int, mean_gap: float):
    """Chunk k of the capacity stream: records with issue times relative to the chunk's start."""
    rng = np.random.Generator(np.random.PCG64([seed, 4, k]))
    replica = rng.integers(0, CAPACITY_REPLICAS, m, dtype=np.uint64)
    lg = rng.integers(7, 17, m, dtype=np.uint64)                     # 128 B ... 64 KiB
    slots = np.uint64(WEIGHT_BYTES) >> lg
    slot = (rng.random(m) * slots.astype(np.float64)).astype(np.uint64)
    slot = np.minimum(slot, slots - np.uint64(1))
    out = np.empty(m, ACCESS_DTYPE)
    out["addr"] = np.uint64(RANGE_BASE) + replica * np.uint64(CAPACITY_SLOT) + (slot << lg)
    out["bytes"] = (np.uint64(1) << lg).astype(np.uint32)
    out["flags"] = 0
    rel = np.cumsum(rng.exponential(mean_gap, m))
    return out, rel


def capacity_chunks(n: int = 200_000_000, seed: int = 0, rho: float = 0.5, profile: str = "nominal",
                    chunk: int = 4_000_000, workers: int | None = None):
    """Yields the capacity-mode stream in issue order, ``chunk`` records at a time.  Chunks are drawn
    from independent substreams (in a thread pool); issue times are chained across chunks."""
    from concurrent.futures import ThreadPoolExecutor
    prof = load_profile(profile, **GEOMETRY["capacity"])
    R = 64 * 8 * 4
    mean_gap = 1.4 * prof["t_read_ns"] / (rho * R)                  # E[pages per read] = 1.4
    sizes = [min(chunk, n - s) for s in range(0, n, chunk)]
    workers = workers or min(32, os.cpu_count() or 1)
    t0 = 0.0
    with ThreadPoolExecutor(workers) as pool:
        pending = []
        it = iter(enumerate(sizes))
        for _ in range(workers + 1):
            nxt = next(it, None)
            if nxt is not None:
                pending.append(pool.submit(_capacity_chunk, seed, nxt[0], nxt[1], mean_gap))
        while pending:
            out, rel = pending.pop(0).result()
            nxt = next(it, None)
            if nxt is not None:
                pending.append(pool.submit(_capacity_chunk, seed, nxt[0], nxt[1], mean_gap))
            out["issue_ns"] = np.floor(rel + t0).astype(np.int64)
            t0 += float(rel[-1])
            yield out


def capacity_mode(n: int = 200_000_000, seed: int = 0, rho: float = 0.5, profile: str = "nominal",
                  out: np.ndarray | None = None) -> Workload:
    prof = load_profile(profile, **GEOMETRY["capacity"])
    acc = out if out is not None else np.empty(n, ACCESS_DTYPE)
    pos = 0
    for part in capacity_chunks(n, seed, rho, profile):
        acc[pos:pos + part.shape[0]] = part
        pos += part.shape[0]
    return Workload("capacity_mode", prof, [(RANGE_BASE, CAPACITY_RANGE, PERM_R | PERM_P, 1, 0, 0)], acc[:n],
                    dict(rho=rho, queues=64 * 8 * 4))


# ---- config 5: long run in 1 ms batches ----------------------------------------------------------------

def timed_batches(w: Workload, horizon_ns: int, window_ns: int = 1_000_000):
    """Repeats ``w`` back to back (each repeat shifted by the stream's span) up to ``horizon_ns`` and
    yields ``(window_index, records)`` for every window, empty ones included."""
    acc = w.acc
    span = int(acc["issue_ns"][-1]) + 1
    n_win = (horizon_ns + window_ns - 1) // window_ns
    rep, base, pos = 0, 0, 0
    for k in range(n_win):
        hi = (k + 1) * window_ns
        parts = []
        while True:
            end = pos + int(np.searchsorted(acc["issue_ns"][pos:], hi - base, side="left"))
            if end > pos:
                p = acc[pos:end].copy(); p["issue_ns"] += base; parts.append(p)
            pos = end
            if pos < acc.shape[0]:
                break
            rep += 1; base = rep * span; pos = 0
            if base >= hi:
                break
        yield k, (np.concatenate(parts) if parts else np.empty(0, ACCESS_DTYPE))


# ---- parity-only mixed stream ---------------------------------------------------------------------------

def mixed_status(n: int = 10_000, seed: int = 0, faults: bool = False, profile: str = "nominal") -> Workload:
    """Two ranges (the second read-only) with gaps, 10 % accesses outside every range, reads and
    programs of mixed sizes, record order shuffled; optionally three fail-closed accesses."""
    prof = load_profile(profile, **GEOMETRY["tiny"])
    rng = np.random.Generator(np.random.PCG64([seed, 6]))
    r0 = (RANGE_BASE, 256 * MIB, PERM_R | PERM_P, 0, 7, 0)
    r1 = (RANGE_BASE + 512 * MIB, 128 * MIB, PERM_R, 0, 9, 256 * MIB)
    where = rng.random(n)
    lg = rng.integers(6, 17, n)
    size = (1 << lg).astype(np.int64) + rng.integers(0, 2, n) * rng.integers(0, 4096, n)
    in0 = where < 0.6
    in1 = (where >= 0.6) & (where < 0.9)
    off0 = (rng.random(n) * (256 * MIB - size)).astype(np.int64)
    off1 = (rng.random(n) * (128 * MIB - size)).astype(np.int64)
    gap = RANGE_BASE + 256 * MIB + (rng.random(n) * (256 * MIB - size)).astype(np.int64)
    addr = np.where(in0, r0[0] + off0, np.where(in1, r1[0] + off1, gap)).astype(np.uint64)
    flags = np.where(in0 & (rng.random(n) < 0.2), 1, 0).astype(np.uint32)
    issue = rng.integers(0, 20_000_000, n, dtype=np.int64)
    issue[rng.integers(0, n, n // 10)] = issue[rng.integers(0, n, n // 10)]          # equal issue times
    acc = _records(addr, issue, size.astype(np.uint32), flags)
    if faults:
        i, j, k = (int(x) for x in rng.choice(n, 3, replace=False))
        acc[i] = (r0[0] + r0[1] - 100, 5, 4096, 0)            # leaves its range
        acc[j] = (r1[0] + 4096, 6, 4096, 1)                   # program to a read-only range
        acc[k] = (r0[0], 7, 0, 0)                             # zero bytes
    return Workload("mixed_status", prof, [r0, r1], acc, dict(faults=faults))


# ---- package floorplan ------------------------------------------------------------------------------------

_CELL = {  # kind: (lateral g W/K, C J/K, G_sink W/K)
    KIND_NONE: (0.03, 5e-5 * 1, 3.6e-4 * 1.0),
    KIND_GPU:  (0.075, 5e-5 * 1, 3.6e-4 * 1.0),
    KIND_HBM:  (0.05, 5e-5 * 3, 3.6e-4 * 0.75),
    KIND_HBF:  (0.05, 5e-5 * 4, 3.6e-4 * 0.5),
}


def _finish_floorplan(kind_of_cell, cell_region, region_kind, region_idle_w, die_region, ext_power_w):
    H, W = kind_of_cell.shape
    g = np.vectorize(lambda k: _CELL[k][0])(kind_of_cell).astype(np.float64)
    Cc = np.vectorize(lambda k: _CELL[k][1])(kind_of_cell)
    Gs = np.vectorize(lambda k: _CELL[k][2])(kind_of_cell)
    Gx = np.zeros((H, W)); Gy = np.zeros((H, W))
    Gx[:, :-1] = 2 * g[:, :-1] * g[:, 1:] / (g[:, :-1] + g[:, 1:])       # series half cells
    Gy[:-1, :] = 2 * g[:-1, :] * g[1:, :] / (g[:-1, :] + g[1:, :])
    return dict(grid_h=H, grid_w=W,
                cell_C=Cc.astype(np.float32).ravel(), cell_Gx=Gx.astype(np.float32).ravel(),
                cell_Gy=Gy.astype(np.float32).ravel(), cell_Gsink=Gs.astype(np.float32).ravel(),
                cell_region=cell_region.astype(np.int32).ravel(), die_region=np.asarray(die_region, np.int32),
                region_kind=np.asarray(region_kind, np.int32), region_idle_w=np.asarray(region_idle_w, np.float32),
                ext_power_w=np.asarray(ext_power_w, np.float32))


def package_floorplan(channels: int = 32, dies: int = 8) -> dict:
    """128x128 cells of 0.25 mm: a GPU die of 7x4 tiles, three HBM stacks and two HBF stacks of
    16 channel blocks each (the paper's three-HBM / two-HBF layout).  All dies of a channel map to
    that channel's block.  External power: 86.6 W over the GPU tiles (the paper's compute-limit
    load), 8 W per HBM stack; HBF idle 5 W per stack."""
    assert channels % 32 == 0, "the package floorplan has 2 HBF stacks x 16 channel blocks"
    H = W = 128
    kind = np.zeros((H, W), np.int64); region = -np.ones((H, W), np.int64)
    region_kind, idle, ext = [], [], []
    for ty in range(7):
        for tx in range(4):
            y0, x0 = 8 + 16 * ty, 32 + 16 * tx
            kind[y0:y0 + 16, x0:x0 + 16] = KIND_GPU; region[y0:y0 + 16, x0:x0 + 16] = len(region_kind)
            region_kind.append(KIND_GPU); idle.append(0.0); ext.append(86.6 / 28)
    for y0 in (8, 48, 88):
        kind[y0:y0 + 32, 4:28] = KIND_HBM; region[y0:y0 + 32, 4:28] = len(region_kind)
        region_kind.append(KIND_HBM); idle.append(0.0); ext.append(8.0)
    first_hbf = len(region_kind)
    for s, y0 in enumerate((8, 72)):
        for b in range(16):
            by, bx = y0 + 12 * (b // 4), 100 + 6 * (b % 4)
            kind[by:by + 12, bx:bx + 6] = KIND_HBF; region[by:by + 12, bx:bx + 6] = len(region_kind)
            region_kind.append(KIND_HBF); idle.append(5.0 / 16); ext.append(0.0)
    die_region = [first_hbf + c % 32 for c in range(channels) for _ in range(dies)]     # channels beyond 32 share blocks
    return _finish_floorplan(kind, region, region_kind, idle, die_region, ext)


def toy_floorplan(h: int, w: int, channels: int, dies: int, seed: int = 0) -> dict:
    """A small irregular floorplan for tests: left part GPU, a HBM strip, HBF channel columns."""
    rng = np.random.Generator(np.random.PCG64([seed, 7]))
    kind = np.zeros((h, w), np.int64); region = -np.ones((h, w), np.int64)
    region_kind, idle, ext = [KIND_GPU, KIND_HBM], [0.0, 0.0], [float(rng.uniform(1, 3)), float(rng.uniform(0.2, 1))]
    kind[1:h - 1, 1:w // 3] = KIND_GPU; region[1:h - 1, 1:w // 3] = 0
    kind[1:h // 2, w // 3 + 1:w // 2] = KIND_HBM; region[1:h // 2, w // 3 + 1:w // 2] = 1
    cols = np.array_split(np.arange(w // 2 + 1, w - 1), channels)
    for c, cs in enumerate(cols):
        assert len(cs) > 0, "grid too narrow for that many channels"
        kind[1:h - 1, cs] = KIND_HBF; region[1:h - 1, cs] = len(region_kind)
        region_kind.append(KIND_HBF); idle.append(0.05); ext.append(0.0)
    die_region = [2 + c for c in range(channels) for _ in range(dies)]
    return _finish_floorplan(kind, region, region_kind, idle, die_region, ext)
