"""ctypes binding of the sequential CPU oracle (``hbfo.c``).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this module.  It shares
nothing with the CUDA library or its binding: the structures below restate ``hbfo.h``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libhbfo.so")

ST_NATIVE, ST_READY, ST_FAULT_PARTIAL, ST_FAULT_PERM, ST_UNSUPPORTED = range(5)
MODE_NORMAL, MODE_LIGHT, MODE_SEVERE, MODE_SHUTDOWN = range(4)
OK, E_INVAL, E_RANGE_OVERLAP, E_RANGE_FULL, E_CAPACITY = 0, -1, -2, -3, -4
E_ACCESS_FAULT, E_THROTTLED, E_LINK_SHUTDOWN = -7, -8, -9

ACCESS_DTYPE = np.dtype([("addr", "<u8"), ("issue_ns", "<i8"), ("bytes", "<u4"), ("flags", "<u4")])
DIE_STATS_DTYPE = np.dtype([(k, "<i8") for k in
                            ("busy_ns", "bytes_read", "bytes_prog", "energy_pj", "n_read", "n_prog")])


class Config(C.Structure):
    _fields_ = [
        ("channels", C.c_uint32), ("dies", C.c_uint32), ("planes", C.c_uint32),
        ("page_bytes", C.c_uint32), ("stripe_bytes", C.c_uint32), ("queue_level", C.c_uint32),
        ("capacity_bytes", C.c_uint64),
        ("t_read_ns", C.c_int64), ("t_prog_ns", C.c_int64),
        ("chan_bytes_per_us", C.c_uint64),
        ("read_granule", C.c_uint32), ("prog_granule", C.c_uint32),
        ("e_cmd_read_pj", C.c_int64), ("e_byte_read_pj", C.c_int64),
        ("e_cmd_prog_pj", C.c_int64), ("e_byte_prog_pj", C.c_int64),
        ("grid_h", C.c_uint32), ("grid_w", C.c_uint32), ("n_sub", C.c_uint32), ("n_regions", C.c_uint32),
        ("ambient_c", C.c_float), ("rtt_c", C.c_float), ("ltt_c", C.c_float), ("stt_c", C.c_float),
        ("shutdown_c", C.c_float),
        ("q_light_ppm", C.c_int64),
        ("cell_C", C.c_void_p), ("cell_Gx", C.c_void_p), ("cell_Gy", C.c_void_p), ("cell_Gsink", C.c_void_p),
        ("cell_region", C.c_void_p), ("die_region", C.c_void_p), ("region_kind", C.c_void_p),
        ("region_idle_w", C.c_void_p),
    ]


class BatchResult(C.Structure):
    _fields_ = [("code", C.c_int32), ("mode", C.c_int32), ("q_ppm", C.c_int64),
                ("n_native", C.c_uint64), ("n_modeled", C.c_uint64), ("n_fault", C.c_uint64),
                ("modeled_ns", C.c_int64), ("service_ns", C.c_int64), ("max_completion_ns", C.c_int64)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


def build(force: bool = False) -> str:
    """Compile ``hbfo.c`` into ``libhbfo.so`` next to it (gcc, -O2) and return the path."""
    src = os.path.join(_HERE, "hbfo.c")
    hdr = os.path.join(_HERE, "hbfo.h")
    if (not force and os.path.exists(_SO)
            and os.path.getmtime(_SO) >= max(os.path.getmtime(src), os.path.getmtime(hdr))):
        return _SO
    tmp = _SO + ".tmp%d" % os.getpid()
    subprocess.check_call(["gcc", "-std=c11", "-O2", "-fPIC", "-shared", "-Wall", "-Wextra", "-o", tmp, src, "-lm"])
    os.replace(tmp, _SO)
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.hbfo_strerror.restype = C.c_char_p
        L.hbfo_euler_limit_ns.restype = C.c_double
        L.hbfo_euler_limit_ns.argtypes = [C.c_void_p]
        L.hbfo_quantise_mk.restype = C.c_int64
        L.hbfo_quantise_mk.argtypes = [C.c_double]
        L.hbfo_next_mode.restype = C.c_int32
        L.hbfo_next_mode.argtypes = [C.c_void_p, C.c_int32, C.c_int64]
        L.hbfo_create.argtypes = [C.POINTER(Config), C.POINTER(C.c_void_p)]
        L.hbfo_destroy.argtypes = [C.c_void_p]
        L.hbfo_register_range.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32,
                                          C.c_uint32, C.c_uint64, C.POINTER(C.c_uint32)]
        L.hbfo_clear_ranges.argtypes = [C.c_void_p]
        L.hbfo_submit_batch.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_void_p]
        L.hbfo_submit_batch_paged.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_void_p]
        L.hbfo_enable_channel_bus.argtypes = [C.c_void_p]
        L.hbfo_get_bus_busy_until.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        L.hbfo_enable_energy_bins.argtypes = [C.c_void_p, C.c_int64, C.c_uint32]
        L.hbfo_get_energy_bins.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.POINTER(C.c_int64)]
        L.hbfo_enable_retention.argtypes = [C.c_void_p, C.POINTER(RetentionConfig)]
        L.hbfo_retention_advance.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
        L.hbfo_retention_decay.argtypes = [C.c_void_p, C.c_int64]
        L.hbfo_get_retention_blocks.argtypes = [C.c_void_p] + [C.c_void_p] * 4 + [C.c_uint64]
        L.hbfo_get_retention_plan.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.POINTER(C.c_uint64)]
        L.hbfo_get_retention_totals.argtypes = [C.c_void_p, C.POINTER(RetentionTotals)]
        L.hbfo_retention_lifetime_s.argtypes = [C.c_void_p, C.c_double]
        L.hbfo_retention_lifetime_s.restype = C.c_double
        L.hbfo_rom_create.argtypes = [C.c_uint32, C.c_uint32, C.c_uint32] + [C.c_void_p] * 6 + [C.POINTER(C.c_void_p)]
        L.hbfo_thermal_step_rom.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_uint32, C.c_void_p]
        L.hbfo_rom_destroy.argtypes = [C.c_void_p]
        L.hbfo_rom_reset.argtypes = [C.c_void_p]
        L.hbfo_rom_step.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p]
        L.hbfo_rom_get_state.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        L.hbfo_last_result.argtypes = [C.c_void_p, C.POINTER(BatchResult)]
        L.hbfo_last_order.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.POINTER(C.c_uint64)]
        L.hbfo_thermal_step.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p]
        L.hbfo_force_mode.argtypes = [C.c_void_p, C.c_int32, C.c_int64]
        L.hbfo_reset.argtypes = [C.c_void_p]
        L.hbfo_get_busy_until.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        L.hbfo_get_pending_energy.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        L.hbfo_get_temps.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        L.hbfo_set_temps.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        L.hbfo_get_mode.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
        L.hbfo_classify.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int32)]
        L.hbfo_decode.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32] + [C.c_void_p] * 7
        L.hbfo_service_terms.argtypes = [C.c_void_p, C.c_uint32, C.c_uint64, C.c_uint32, C.c_int64] + [C.c_void_p] * 4
        _lib = L
    return _lib


_SCALARS = ("channels", "dies", "planes", "page_bytes", "stripe_bytes", "queue_level", "capacity_bytes",
            "t_read_ns", "t_prog_ns", "chan_bytes_per_us", "read_granule", "prog_granule",
            "e_cmd_read_pj", "e_byte_read_pj", "e_cmd_prog_pj", "e_byte_prog_pj",
            "grid_h", "grid_w", "n_sub", "n_regions", "ambient_c", "rtt_c", "ltt_c", "stt_c", "shutdown_c",
            "q_light_ppm")
_ARRAYS = (("cell_C", np.float32), ("cell_Gx", np.float32), ("cell_Gy", np.float32), ("cell_Gsink", np.float32),
           ("cell_region", np.int32), ("die_region", np.int32), ("region_kind", np.int32),
           ("region_idle_w", np.float32))


class RetentionConfig(C.Structure):
    _fields_ = [("pages_per_block", C.c_uint32), ("blocks_per_plane", C.c_uint32), ("blocks_per_zone", C.c_uint32),
                ("max_pec", C.c_uint32), ("disturb_limit", C.c_uint32), ("pad", C.c_uint32),
                ("l_ref_s", C.c_double), ("t_ref_c", C.c_double), ("ea_ev", C.c_double),
                ("accel", C.c_double), ("lead_threshold", C.c_double)]


class RetentionTotals(C.Structure):
    _fields_ = [(k, C.c_uint64) for k in ("n_blocks", "planned", "claimed", "decayed", "commits", "worn_blocks",
                                          "waiting_blocks")] + [("epoch", C.c_uint32), ("pad", C.c_uint32)]


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__("hbfo: %s (%d)" % (lib().hbfo_strerror(code).decode(), code))
        self.code = code


class Oracle:
    """One oracle context.  ``profile`` is a dict of the scalar fields of ``hbfo_config_t``;
    ``floorplan`` (optional) a dict of the thermal arrays."""

    def __init__(self, profile: dict, floorplan: dict | None = None):
        cfg = Config()
        for k in _SCALARS:
            if k in profile:
                setattr(cfg, k, profile[k])
        self._keep = []
        if floorplan is not None:
            for k, dt in _ARRAYS:
                arr = np.ascontiguousarray(floorplan[k], dtype=dt)
                self._keep.append(arr)
                setattr(cfg, k, arr.ctypes.data)
            cfg.grid_h, cfg.grid_w = floorplan["grid_h"], floorplan["grid_w"]
            cfg.n_regions = len(floorplan["region_kind"])
        self.cfg = cfg
        self.n_dies = cfg.channels * cfg.dies
        self.n_channels = cfg.channels
        self.n_queues = self.n_dies * (cfg.planes if cfg.queue_level == 0 else 1)
        self.n_cells = cfg.grid_h * cfg.grid_w if floorplan is not None else 0
        h = C.c_void_p()
        rc = lib().hbfo_create(C.byref(cfg), C.byref(h))
        if rc != 0:
            raise OracleError(rc)
        self._h = h

    def close(self):
        if self._h:
            lib().hbfo_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def register_range(self, base, length, perms=3, kind=0, stream_tag=0, media_offset=0, check=True):
        rid = C.c_uint32()
        rc = lib().hbfo_register_range(self._h, base, length, perms, kind, stream_tag, media_offset, C.byref(rid))
        if rc != 0:
            if check:
                raise OracleError(rc)
            return rc
        return rid.value

    def clear_ranges(self):
        lib().hbfo_clear_ranges(self._h)

    def submit(self, acc: np.ndarray, check=True, paged=False):
        """Returns (code, completion, stall, status, die_stats).  paged: every page of an access is a request of its own."""
        acc = np.ascontiguousarray(acc, dtype=ACCESS_DTYPE)
        n = acc.shape[0]
        comp = np.empty(n, np.int64)
        stall = np.empty(n, np.int64)
        status = np.empty(n, np.uint8)
        ds = np.zeros(self.n_dies, DIE_STATS_DTYPE)
        fn = lib().hbfo_submit_batch_paged if paged else lib().hbfo_submit_batch
        rc = fn(self._h, acc.ctypes.data, n, comp.ctypes.data, stall.ctypes.data, status.ctypes.data, ds.ctypes.data)
        if check and rc != 0:
            raise OracleError(rc)
        return rc, comp, stall, status, ds

    def thermal_step_rom(self, rom, output_kind, dt_ns, ext_power_w=None):
        """One thermal step on the reduced-order model ``rom`` (a ``Rom``); returns hot[3]."""
        hot = np.empty(3, np.float64)
        kinds = np.ascontiguousarray(output_kind, np.int32)
        if ext_power_w is None:
            p, n = None, 0
        else:
            ext = np.ascontiguousarray(ext_power_w, np.float32)
            p, n = ext.ctypes.data, ext.shape[0]
        rc = lib().hbfo_thermal_step_rom(self._h, rom._h, kinds.ctypes.data, dt_ns, p, n, hot.ctypes.data)
        if rc != 0:
            raise OracleError(rc)
        return hot

    # ---- retention, refresh and wear (Design D4) ----
    def enable_retention(self, **kw):
        """Keyword arguments are the fields of ``hbfo_retention_config_t``."""
        cfg = RetentionConfig()
        for k, v in kw.items():
            setattr(cfg, k, v)
        rc = lib().hbfo_enable_retention(self._h, C.byref(cfg))
        if rc != 0:
            raise OracleError(rc)
        self._ret_blocks = self.n_dies * self.cfg.planes * cfg.blocks_per_plane

    def retention_advance(self, dt_ns, region_temp_c=None):
        t = None if region_temp_c is None else np.ascontiguousarray(region_temp_c, np.float64)
        rc = lib().hbfo_retention_advance(self._h, dt_ns, None if t is None else t.ctypes.data)
        if rc != 0:
            raise OracleError(rc)

    def retention_decay(self, idle_ns):
        rc = lib().hbfo_retention_decay(self._h, idle_ns)
        if rc != 0:
            raise OracleError(rc)

    def retention_blocks(self) -> dict:
        nb = self._ret_blocks
        out = {"damage": np.zeros(nb, np.float64), "disturb": np.zeros(nb, np.uint32), "pec": np.zeros(nb, np.uint32),
               "epoch": np.zeros(nb, np.uint32)}
        rc = lib().hbfo_get_retention_blocks(self._h, out["damage"].ctypes.data, out["disturb"].ctypes.data,
                                             out["pec"].ctypes.data, out["epoch"].ctypes.data, nb)
        if rc != 0:
            raise OracleError(rc)
        return out

    def retention_plan(self) -> np.ndarray:
        cnt = C.c_uint64()
        lib().hbfo_get_retention_plan(self._h, None, 0, C.byref(cnt))
        out = np.zeros(cnt.value, np.uint32)
        rc = lib().hbfo_get_retention_plan(self._h, out.ctypes.data, out.size, C.byref(cnt))
        if rc != 0:
            raise OracleError(rc)
        return out

    def retention_totals(self) -> dict:
        t = RetentionTotals()
        rc = lib().hbfo_get_retention_totals(self._h, C.byref(t))
        if rc != 0:
            raise OracleError(rc)
        return {k: getattr(t, k) for k, _ in t._fields_ if k != "pad"}

    def retention_lifetime_s(self, temp_c) -> float:
        return lib().hbfo_retention_lifetime_s(self._h, float(temp_c))

    def enable_channel_bus(self):
        rc = lib().hbfo_enable_channel_bus(self._h)
        if rc != 0:
            raise OracleError(rc)

    def bus_busy_until(self) -> np.ndarray:
        out = np.zeros(self.n_channels, np.int64)
        rc = lib().hbfo_get_bus_busy_until(self._h, out.ctypes.data, out.size)
        if rc != 0:
            raise OracleError(rc)
        return out

    def enable_energy_bins(self, bin_ns: int, n_bins: int):
        rc = lib().hbfo_enable_energy_bins(self._h, bin_ns, n_bins)
        if rc != 0:
            raise OracleError(rc)
        self._n_bins = n_bins

    def energy_bins(self):
        """(first_bin, array [n_bins][n_dies] of pJ): row k is bin first_bin + k."""
        out = np.zeros((self._n_bins, self.n_dies), np.int64)
        first = C.c_int64()
        rc = lib().hbfo_get_energy_bins(self._h, out.ctypes.data, out.size, C.byref(first))
        if rc != 0:
            raise OracleError(rc)
        return first.value, out

    def last_result(self) -> dict:
        r = BatchResult()
        lib().hbfo_last_result(self._h, C.byref(r))
        return r.as_dict()

    def last_order(self) -> np.ndarray:
        cnt = C.c_uint64()
        lib().hbfo_last_order(self._h, None, 0, C.byref(cnt))
        out = np.empty(cnt.value, np.uint32)
        lib().hbfo_last_order(self._h, out.ctypes.data, cnt.value, C.byref(cnt))
        return out

    def thermal_step(self, dt_ns, ext_power_w=None, want_temps=False):
        """Returns (hot[3], temps or None)."""
        hot = np.empty(3, np.float64)
        temps = np.empty(self.n_cells, np.float64) if want_temps else None
        if ext_power_w is None:
            p, n = None, 0
        else:
            ext = np.ascontiguousarray(ext_power_w, np.float32)
            p, n = ext.ctypes.data, ext.shape[0]
        rc = lib().hbfo_thermal_step(self._h, dt_ns, p, n, temps.ctypes.data if want_temps else None,
                                     hot.ctypes.data)
        if rc != 0:
            raise OracleError(rc)
        return hot, temps

    def force_mode(self, mode, q_ppm):
        rc = lib().hbfo_force_mode(self._h, mode, q_ppm)
        if rc != 0:
            raise OracleError(rc)

    def reset(self):
        lib().hbfo_reset(self._h)

    def busy_until(self) -> np.ndarray:
        out = np.empty(self.n_queues, np.int64)
        lib().hbfo_get_busy_until(self._h, out.ctypes.data, out.shape[0])
        return out

    def pending_energy(self) -> np.ndarray:
        out = np.empty(self.n_dies, np.int64)
        lib().hbfo_get_pending_energy(self._h, out.ctypes.data, out.shape[0])
        return out

    def temps(self) -> np.ndarray:
        out = np.empty(self.n_cells, np.float64)
        rc = lib().hbfo_get_temps(self._h, out.ctypes.data, out.shape[0])
        if rc != 0:
            raise OracleError(rc)
        return out

    def set_temps(self, t):
        t = np.ascontiguousarray(t, np.float64)
        rc = lib().hbfo_set_temps(self._h, t.ctypes.data, t.shape[0])
        if rc != 0:
            raise OracleError(rc)

    def mode(self):
        m, q = C.c_int32(), C.c_int64()
        lib().hbfo_get_mode(self._h, C.byref(m), C.byref(q))
        return m.value, q.value

    def euler_limit_ns(self) -> float:
        return lib().hbfo_euler_limit_ns(self._h)

    def classify(self, addr, bytes_, flags=0, issue_ns=0):
        a = np.zeros(1, ACCESS_DTYPE)
        a["addr"], a["bytes"], a["flags"], a["issue_ns"] = addr, bytes_, flags, issue_ns
        rid = C.c_int32()
        st = lib().hbfo_classify(self._h, a.ctypes.data, C.byref(rid))
        return st, rid.value

    def decode(self, off, bytes_):
        ch, di, pl, qu = C.c_uint32(), C.c_uint32(), C.c_uint32(), C.c_uint32()
        row, page, npg = C.c_uint64(), C.c_uint64(), C.c_uint64()
        lib().hbfo_decode(self._h, off, bytes_, C.addressof(ch), C.addressof(di), C.addressof(pl),
                          C.addressof(row), C.addressof(page), C.addressof(npg), C.addressof(qu))
        return dict(channel=ch.value, die=di.value, plane=pl.value, row=row.value, page=page.value,
                    npages=npg.value, queue=qu.value)

    def service_terms(self, bytes_, npages, op, q_ppm=1000000):
        cb, xf, s, e = C.c_int64(), C.c_int64(), C.c_int64(), C.c_int64()
        rc = lib().hbfo_service_terms(self._h, bytes_, npages, op, q_ppm, C.addressof(cb), C.addressof(xf),
                                      C.addressof(s), C.addressof(e))
        if rc != 0:
            raise OracleError(rc)
        return dict(charged_bytes=cb.value, xfer_ns=xf.value, s_ns=s.value, energy_pj=e.value)

    def next_mode(self, mode, t_hot_mk):
        return lib().hbfo_next_mode(self._h, mode, t_hot_mk)


def quantise_mk(t_c: float) -> int:
    return lib().hbfo_quantise_mk(t_c)


class Rom:
    """Reduced-order thermal model (Eq. 2) stepped in double by plain loops."""

    def __init__(self, A, B, C_, D=None, b=None, d=None):
        A = np.ascontiguousarray(A, np.float64); B = np.ascontiguousarray(B, np.float64); C_ = np.ascontiguousarray(C_, np.float64)
        self.n, self.m, self.o = A.shape[0], B.shape[1], C_.shape[0]
        opt = lambda v, shape: None if v is None else np.ascontiguousarray(np.broadcast_to(np.asarray(v, np.float64), shape))
        D, b, d = opt(D, (self.o, self.m)), opt(b, (self.n,)), opt(d, (self.o,))
        ptr = lambda v: None if v is None else v.ctypes.data
        h = C.c_void_p()
        rc = lib().hbfo_rom_create(self.n, self.m, self.o, ptr(A), ptr(B), ptr(b), ptr(C_), ptr(D), ptr(d), C.byref(h))
        if rc != 0:
            raise OracleError(rc)
        self._h = h

    def __del__(self):
        try:
            if getattr(self, "_h", None):
                lib().hbfo_rom_destroy(self._h); self._h = None
        except Exception:
            pass

    def reset(self):
        lib().hbfo_rom_reset(self._h)

    def step(self, power):
        """power [n_steps][n_inputs] -> temperatures [n_steps][n_outputs]"""
        p = np.ascontiguousarray(np.atleast_2d(power), np.float64)
        out = np.empty((p.shape[0], self.o), np.float64)
        rc = lib().hbfo_rom_step(self._h, p.ctypes.data, p.shape[0], out.ctypes.data)
        if rc != 0:
            raise OracleError(rc)
        return out

    def state(self):
        x = np.empty(self.n, np.float64)
        lib().hbfo_rom_get_state(self._h, x.ctypes.data, self.n)
        return x
