"""Thin ctypes binding of ``libhbf.so`` (``include/hbf.h``): argument marshalling only.

Every step of the service model runs in the library's CUDA kernels.  PyTorch is used for device
memory and streams.  There is no CPU fallback: if the library has not been built, or no CUDA device
is present, the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libhbf.so")

OK, E_INVAL, E_RANGE_OVERLAP, E_RANGE_FULL, E_CAPACITY, E_WORKSPACE, E_CUDA = 0, -1, -2, -3, -4, -5, -6
E_ACCESS_FAULT, E_THROTTLED, E_LINK_SHUTDOWN, E_TIMEOUT, E_NOMEM = -7, -8, -9, -10, -11
ST_NATIVE, ST_READY, ST_FAULT_PARTIAL, ST_FAULT_PERM, ST_UNSUPPORTED = range(5)
MODE_NORMAL, MODE_LIGHT, MODE_SEVERE, MODE_SHUTDOWN = range(4)
KIND_NONE, KIND_GPU, KIND_HBM, KIND_HBF = range(4)
PATH_AUTO, PATH_SORT, PATH_INORDER, PATH_SORT_FULL = range(4)

ACCESS_DTYPE = np.dtype([("addr", "<u8"), ("issue_ns", "<i8"), ("bytes", "<u4"), ("flags", "<u4")])
DIE_STATS_DTYPE = np.dtype([(k, "<i8") for k in
                            ("busy_ns", "bytes_read", "bytes_prog", "energy_pj", "n_read", "n_prog")])

EXPORTS = ("hbf_create", "hbf_destroy", "hbf_register_range", "hbf_clear_ranges", "hbf_workspace_bytes",
           "hbf_submit_batch", "hbf_last_result", "hbf_thermal_step", "hbf_force_mode", "hbf_get_mode",
           "hbf_reset", "hbf_set_path", "hbf_set_tile_balance", "hbf_get_tile_times", "hbf_set_head_entries", "hbf_get_state", "hbf_set_state", "hbf_get_busy_until",
           "hbf_get_pending_energy", "hbf_get_temps", "hbf_euler_limit_ns", "hbf_queue_order", "hbf_strerror",
           "hbf_set_profiling", "hbf_get_profile", "hbf_kernel_launches", "hbf_euler_substeps_static", "hbf_set_thermal_path",
           "hbf_workspace_bytes_paged", "hbf_submit_batch_paged", "hbf_submit_host", "hbf_debug_wait_test",
           "hbf_enable_energy_bins", "hbf_get_energy_bins", "hbf_enable_channel_bus", "hbf_get_bus_busy_until",
           "hbf_rom_create", "hbf_rom_destroy", "hbf_rom_reset", "hbf_rom_step", "hbf_rom_get_state",
           "hbf_attach_rom", "hbf_get_rom_temps",
           "hbf_enable_retention", "hbf_retention_advance", "hbf_retention_decay", "hbf_get_retention_blocks",
           "hbf_get_retention_plan", "hbf_get_retention_totals")
STATIC_MAX_CELLS = 65536
PROF_STAGES = ("begin", "classify", "plan_hist", "sort", "scan", "finish", "inorder", "thermal")


class hbf_retention_config_t(C.Structure):
    _fields_ = [("pages_per_block", C.c_uint32), ("blocks_per_plane", C.c_uint32), ("blocks_per_zone", C.c_uint32),
                ("max_pec", C.c_uint32), ("disturb_limit", C.c_uint32), ("pad", C.c_uint32),
                ("l_ref_s", C.c_double), ("t_ref_c", C.c_double), ("ea_ev", C.c_double),
                ("accel", C.c_double), ("lead_threshold", C.c_double)]


class hbf_retention_totals_t(C.Structure):
    _fields_ = [(k, C.c_uint64) for k in ("n_blocks", "planned", "claimed", "decayed", "commits", "worn_blocks",
                                          "waiting_blocks")] + [("epoch", C.c_uint32), ("pad", C.c_uint32)]


class hbf_config_t(C.Structure):
    _fields_ = [
        ("channels", C.c_uint32), ("dies", C.c_uint32), ("planes", C.c_uint32),
        ("page_bytes", C.c_uint32), ("stripe_bytes", C.c_uint32), ("queue_level", C.c_uint32),
        ("capacity_bytes", C.c_uint64),
        ("t_read_ns", C.c_int64), ("t_prog_ns", C.c_int64), ("chan_bytes_per_us", C.c_uint64),
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


class hbf_batch_result_t(C.Structure):
    _fields_ = [("code", C.c_int32), ("mode", C.c_int32), ("q_ppm", C.c_int64),
                ("n_native", C.c_uint64), ("n_modeled", C.c_uint64), ("n_fault", C.c_uint64),
                ("modeled_ns", C.c_int64), ("service_ns", C.c_int64), ("max_completion_ns", C.c_int64)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


_lib = None


def library_path() -> str:
    return _SO


def lib():
    """The loaded CUDA library.  Raises if it has not been built (python -m paper_2609_09800_b200.build)."""
    global _lib
    if _lib is None:
        path = os.environ.get("HBF_LIBRARY", _SO)          # an explicitly chosen build of the same library
        if not os.path.exists(path):
            raise RuntimeError("libhbf.so is missing: build it with `python -m paper_2609_09800_b200.build` "
                               "(nvcc, sm_100a); there is no CPU fallback")
        L = C.CDLL(path)
        vp, u64, u32, i64, i32 = C.c_void_p, C.c_uint64, C.c_uint32, C.c_int64, C.c_int32
        L.hbf_create.argtypes = [C.POINTER(hbf_config_t), vp, C.POINTER(vp)]
        L.hbf_destroy.argtypes = [vp]
        L.hbf_register_range.argtypes = [vp, u64, u64, u32, u32, u32, u64, C.POINTER(u32)]
        L.hbf_clear_ranges.argtypes = [vp]
        L.hbf_workspace_bytes.argtypes = [vp, u64]
        L.hbf_workspace_bytes.restype = C.c_size_t
        L.hbf_submit_batch.argtypes = [vp, vp, u64, vp, vp, vp, vp, vp, C.c_size_t]
        L.hbf_debug_wait_test.argtypes = [vp, u32, u32, u32]
        L.hbf_submit_host.argtypes = [vp, vp, u64, vp, vp, vp, u64, C.POINTER(hbf_batch_result_t)]
        L.hbf_workspace_bytes_paged.argtypes = [vp, u64, u64]
        L.hbf_workspace_bytes_paged.restype = C.c_size_t
        L.hbf_submit_batch_paged.argtypes = [vp, vp, u64, u64, vp, vp, vp, vp, vp, C.c_size_t]
        L.hbf_enable_channel_bus.argtypes = [vp]
        L.hbf_get_bus_busy_until.argtypes = [vp, vp, u64]
        L.hbf_enable_energy_bins.argtypes = [vp, i64, u32]
        L.hbf_enable_retention.argtypes = [vp, C.POINTER(hbf_retention_config_t)]
        L.hbf_retention_advance.argtypes = [vp, i64, vp]
        L.hbf_retention_decay.argtypes = [vp, i64]
        L.hbf_get_retention_blocks.argtypes = [vp, vp, vp, vp, vp, u64]
        L.hbf_get_retention_plan.argtypes = [vp, vp, u64, C.POINTER(u64)]
        L.hbf_get_retention_totals.argtypes = [vp, C.POINTER(hbf_retention_totals_t)]
        L.hbf_get_energy_bins.argtypes = [vp, vp, u64, C.POINTER(i64)]
        L.hbf_rom_create.argtypes = [u32, u32, u32, vp, vp, vp, vp, vp, vp, vp, C.POINTER(vp)]
        L.hbf_attach_rom.argtypes = [vp, vp, vp, i64]
        L.hbf_get_rom_temps.argtypes = [vp, vp, u64]
        L.hbf_rom_destroy.argtypes = [vp]
        L.hbf_rom_reset.argtypes = [vp]
        L.hbf_rom_step.argtypes = [vp, vp, u32, vp]
        L.hbf_rom_get_state.argtypes = [vp, vp, u64]
        L.hbf_last_result.argtypes = [vp, C.POINTER(hbf_batch_result_t)]
        L.hbf_thermal_step.argtypes = [vp, i64, vp, u32, vp, vp]
        L.hbf_force_mode.argtypes = [vp, i32, i64]
        L.hbf_get_mode.argtypes = [vp, C.POINTER(i32), C.POINTER(i64)]
        L.hbf_reset.argtypes = [vp]
        L.hbf_set_path.argtypes = [vp, i32]
        L.hbf_set_tile_balance.argtypes = [vp, i32]
        L.hbf_set_head_entries.argtypes = [vp, u32]
        L.hbf_get_tile_times.argtypes = [vp, vp, vp, C.c_uint32, vp]
        L.hbf_set_thermal_path.argtypes = [vp, i32]
        L.hbf_get_state.argtypes = [vp, vp, C.POINTER(C.c_size_t)]
        L.hbf_set_state.argtypes = [vp, vp, C.c_size_t]
        L.hbf_get_busy_until.argtypes = [vp, vp, u64]
        L.hbf_get_pending_energy.argtypes = [vp, vp, u64]
        L.hbf_get_temps.argtypes = [vp, vp, u64]
        L.hbf_euler_limit_ns.argtypes = [vp]
        L.hbf_euler_limit_ns.restype = C.c_double
        L.hbf_queue_order.argtypes = [vp, vp, u64, vp, C.POINTER(u64)]
        L.hbf_set_profiling.argtypes = [vp, C.c_int]
        L.hbf_get_profile.argtypes = [vp, vp, u32]
        L.hbf_kernel_launches.argtypes = []
        L.hbf_kernel_launches.restype = u64
        L.hbf_euler_substeps_static.argtypes = [vp, vp, vp, vp, vp, vp, vp, u32, u32, u32, C.c_float, vp]
        L.hbf_strerror.argtypes = [C.c_int]
        L.hbf_strerror.restype = C.c_char_p
        _lib = L
    return _lib


def kernel_launches() -> int:
    return lib().hbf_kernel_launches()


def euler_substeps_static(d_cell_C, d_cell_Gx, d_cell_Gy, d_cell_Gsink, d_cell_power_w, d_theta, d_comp,
                          grid_h, grid_w, n_sub, dt_sub_s, stream=None) -> int:
    """``hbf_euler_substeps_static``: advances ``d_theta`` (torch CUDA float32 tensors throughout) in place
    using the scratch array built into the library; allocates nothing.  Returns the C return code."""
    import torch
    st = stream if stream is not None else torch.cuda.current_stream()
    return lib().hbf_euler_substeps_static(_ptr(d_cell_C), _ptr(d_cell_Gx), _ptr(d_cell_Gy), _ptr(d_cell_Gsink),
                                           _ptr(d_cell_power_w), _ptr(d_theta), _ptr(d_comp), grid_h, grid_w, n_sub,
                                           dt_sub_s, C.c_void_p(st.cuda_stream))


class HbfError(RuntimeError):
    def __init__(self, code, what=""):
        super().__init__("%s: %s (%d)" % (what or "hbf", lib().hbf_strerror(code).decode(), code))
        self.code = code


_SCALARS = ("channels", "dies", "planes", "page_bytes", "stripe_bytes", "queue_level", "capacity_bytes",
            "t_read_ns", "t_prog_ns", "chan_bytes_per_us", "read_granule", "prog_granule",
            "e_cmd_read_pj", "e_byte_read_pj", "e_cmd_prog_pj", "e_byte_prog_pj",
            "grid_h", "grid_w", "n_sub", "n_regions", "ambient_c", "rtt_c", "ltt_c", "stt_c", "shutdown_c",
            "q_light_ppm")
_ARRAYS = (("cell_C", np.float32), ("cell_Gx", np.float32), ("cell_Gy", np.float32), ("cell_Gsink", np.float32),
           ("cell_region", np.int32), ("die_region", np.int32), ("region_kind", np.int32),
           ("region_idle_w", np.float32))


def make_config(profile: dict, floorplan: dict | None = None):
    """Fills an ``hbf_config_t`` from a profile dict (scalars) and a floorplan dict (host arrays).
    Returns (config, keepalive list)."""
    cfg = hbf_config_t()
    for k in _SCALARS:
        if k in profile:
            setattr(cfg, k, profile[k])
    keep = []
    if floorplan is not None:
        for k, dt in _ARRAYS:
            arr = np.ascontiguousarray(floorplan[k], dtype=dt)
            keep.append(arr)
            setattr(cfg, k, arr.ctypes.data)
        cfg.grid_h, cfg.grid_w = floorplan["grid_h"], floorplan["grid_w"]
        cfg.n_regions = len(floorplan["region_kind"])
    return cfg, keep


def _ptr(t):
    return None if t is None else t.data_ptr()


class Context:
    """One ``hbf_ctx``.  Methods carry the C function's name without the ``hbf_`` prefix and take torch
    CUDA tensors where the C function takes device pointers."""

    def __init__(self, profile: dict, floorplan: dict | None = None, stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("hbf needs a CUDA device; there is no CPU fallback")
        self._torch = torch
        cfg, keep = make_config(profile, floorplan)
        self.n_dies = cfg.channels * cfg.dies
        self.n_channels = cfg.channels
        self.n_planes = cfg.planes
        self.n_queues = self.n_dies * (cfg.planes if cfg.queue_level == 0 else 1)
        self.n_cells = cfg.grid_h * cfg.grid_w if floorplan is not None else 0
        self.n_regions = cfg.n_regions if floorplan is not None else 0
        self.ambient_c = float(cfg.ambient_c)
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        h = C.c_void_p()
        rc = lib().hbf_create(C.byref(cfg), C.c_void_p(self.stream.cuda_stream), C.byref(h))
        if rc != 0:
            raise HbfError(rc, "hbf_create")
        self._h = h
        self._ws = None

    def destroy(self):
        if getattr(self, "_h", None):
            lib().hbf_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # ---- ranges -------------------------------------------------------------------------------
    def register_range(self, base, length, perms=3, kind=0, stream_tag=0, media_offset=0, check=True):
        rid = C.c_uint32()
        rc = lib().hbf_register_range(self._h, base, length, perms, kind, stream_tag, media_offset, C.byref(rid))
        if rc != 0:
            if check:
                raise HbfError(rc, "hbf_register_range")
            return rc
        return rid.value

    def clear_ranges(self):
        return lib().hbf_clear_ranges(self._h)

    # ---- batches ------------------------------------------------------------------------------
    def workspace_bytes(self, n: int) -> int:
        return lib().hbf_workspace_bytes(self._h, n)

    def workspace(self, n: int):
        """A cached device scratch tensor large enough for a batch of n."""
        need = self.workspace_bytes(n)
        if self._ws is None or self._ws.numel() < need:
            self._ws = self._torch.empty(need, dtype=self._torch.uint8, device="cuda")
        return self._ws

    def submit_batch(self, d_acc, n, d_completion, d_stall, d_status=None, d_die_stats=None, d_workspace=None):
        ws = d_workspace if d_workspace is not None else self.workspace(n)
        return lib().hbf_submit_batch(self._h, _ptr(d_acc), n, _ptr(d_completion), _ptr(d_stall), _ptr(d_status),
                                      _ptr(d_die_stats), _ptr(ws), ws.numel() * ws.element_size())

    def workspace_bytes_paged(self, n: int, parts_capacity: int) -> int:
        return lib().hbf_workspace_bytes_paged(self._h, n, parts_capacity)

    def submit_batch_paged(self, d_acc, n, parts_capacity, d_completion, d_stall, d_status=None, d_die_stats=None,
                           d_workspace=None):
        """Page-granular submit: every page of an access is queued on its own (see hbf_submit_batch_paged)."""
        if d_workspace is None:
            need = self.workspace_bytes_paged(n, parts_capacity)
            if self._ws is None or self._ws.numel() < need:
                self._ws = self._torch.empty(need, dtype=self._torch.uint8, device="cuda")
            d_workspace = self._ws
        return lib().hbf_submit_batch_paged(self._h, _ptr(d_acc), n, parts_capacity, _ptr(d_completion), _ptr(d_stall),
                                            _ptr(d_status), _ptr(d_die_stats), _ptr(d_workspace),
                                            d_workspace.numel() * d_workspace.element_size())

    def attach_rom(self, rom, output_kind=None, dt_ns=0):
        """Thermal steps on a reduced-order model (a ``Rom`` created on this context's stream) instead of the grid;
        ``attach_rom(None)`` goes back to the grid."""
        if rom is None:
            rc = lib().hbf_attach_rom(self._h, None, None, 0)
        else:
            kinds = np.ascontiguousarray(output_kind, np.int32)
            rc = lib().hbf_attach_rom(self._h, rom._h, kinds.ctypes.data, dt_ns)
        if rc != 0:
            raise HbfError(rc, "hbf_attach_rom")
        self._rom = rom                                       # keeps the model alive while it is attached

    def get_rom_temps(self):
        out = np.zeros(self._rom.o, np.float64)
        rc = lib().hbf_get_rom_temps(self._h, out.ctypes.data, out.size)
        if rc != 0:
            raise HbfError(rc, "hbf_get_rom_temps")
        return out

    # ---- retention, refresh and wear (Design D4) ----
    def enable_retention(self, **kw):
        """Keyword arguments are the fields of ``hbf_retention_config_t``."""
        cfg = hbf_retention_config_t()
        for k, v in kw.items():
            setattr(cfg, k, v)
        rc = lib().hbf_enable_retention(self._h, C.byref(cfg))
        if rc != 0:
            raise HbfError(rc, "hbf_enable_retention")
        self._ret_blocks = self.n_dies * self.n_planes * cfg.blocks_per_plane

    def retention_advance(self, dt_ns, region_temp_c=None):
        t = None if region_temp_c is None else np.ascontiguousarray(region_temp_c, np.float64)
        rc = lib().hbf_retention_advance(self._h, dt_ns, None if t is None else t.ctypes.data)
        if rc != 0:
            raise HbfError(rc, "hbf_retention_advance")

    def retention_decay(self, idle_ns):
        rc = lib().hbf_retention_decay(self._h, idle_ns)
        if rc != 0:
            raise HbfError(rc, "hbf_retention_decay")

    def retention_blocks(self) -> dict:
        nb = self._ret_blocks
        out = {"damage": np.zeros(nb, np.float64), "disturb": np.zeros(nb, np.uint32), "pec": np.zeros(nb, np.uint32),
               "epoch": np.zeros(nb, np.uint32)}
        rc = lib().hbf_get_retention_blocks(self._h, out["damage"].ctypes.data, out["disturb"].ctypes.data,
                                            out["pec"].ctypes.data, out["epoch"].ctypes.data, nb)
        if rc != 0:
            raise HbfError(rc, "hbf_get_retention_blocks")
        return out

    def retention_plan(self) -> np.ndarray:
        cnt = C.c_uint64()
        rc = lib().hbf_get_retention_plan(self._h, None, 0, C.byref(cnt))
        if rc != 0:
            raise HbfError(rc, "hbf_get_retention_plan")
        out = np.zeros(cnt.value, np.uint32)
        rc = lib().hbf_get_retention_plan(self._h, out.ctypes.data, out.size, C.byref(cnt))
        if rc != 0:
            raise HbfError(rc, "hbf_get_retention_plan")
        return out

    def retention_totals(self) -> dict:
        t = hbf_retention_totals_t()
        rc = lib().hbf_get_retention_totals(self._h, C.byref(t))
        if rc != 0:
            raise HbfError(rc, "hbf_get_retention_totals")
        return {k: getattr(t, k) for k, _ in t._fields_ if k != "pad"}

    def enable_channel_bus(self):
        rc = lib().hbf_enable_channel_bus(self._h)
        if rc != 0:
            raise HbfError(rc, "hbf_enable_channel_bus")
        self._ws = None                                      # the workspace grows once the stage is on

    def get_bus_busy_until(self):
        out = np.zeros(self.n_channels, np.int64)
        rc = lib().hbf_get_bus_busy_until(self._h, out.ctypes.data, out.size)
        if rc != 0:
            raise HbfError(rc, "hbf_get_bus_busy_until")
        return out

    def enable_energy_bins(self, bin_ns: int, n_bins: int):
        rc = lib().hbf_enable_energy_bins(self._h, bin_ns, n_bins)
        if rc != 0:
            raise HbfError(rc, "hbf_enable_energy_bins")
        self._n_bins = n_bins

    def energy_bins(self):
        """(first_bin, array [n_bins][n_dies] of pJ): row k is bin first_bin + k."""
        out = np.zeros((self._n_bins, self.n_dies), np.int64)
        first = C.c_int64()
        rc = lib().hbf_get_energy_bins(self._h, out.ctypes.data, out.size, C.byref(first))
        if rc != 0:
            raise HbfError(rc, "hbf_get_energy_bins")
        return first.value, out

    def last_result(self) -> dict:
        r = hbf_batch_result_t()
        lib().hbf_last_result(self._h, C.byref(r))
        return r.as_dict()

    def queue_order(self, n, d_workspace=None):
        ws = d_workspace if d_workspace is not None else self.workspace(n)
        out = self._torch.empty(max(n, 1), dtype=self._torch.int32, device="cuda")
        cnt = C.c_uint64()
        rc = lib().hbf_queue_order(self._h, _ptr(ws), n, _ptr(out), C.byref(cnt))
        if rc != 0:
            raise HbfError(rc, "hbf_queue_order")
        return out[:cnt.value].cpu().numpy().view(np.uint32)

    def set_path(self, path: int):
        rc = lib().hbf_set_path(self._h, path)
        if rc != 0:
            raise HbfError(rc, "hbf_set_path")

    def tile_times(self):
        """(records, ns) per tile of the last batch that filled a wave of the device; empty arrays when there was none."""
        cnt = C.c_uint32()
        rc = lib().hbf_get_tile_times(self._h, None, None, 0, C.byref(cnt))
        if rc != 0:
            raise HbfError(rc, "hbf_get_tile_times")
        rec = np.zeros(cnt.value, np.uint32); ns = np.zeros(cnt.value, np.uint32)
        if cnt.value:
            rc = lib().hbf_get_tile_times(self._h, rec.ctypes.data, ns.ctypes.data, cnt.value, C.byref(cnt))
            if rc != 0:
                raise HbfError(rc, "hbf_get_tile_times")
        return rec, ns

    def set_head_entries(self, entries: int):
        rc = lib().hbf_set_head_entries(self._h, int(entries))
        if rc != 0:
            raise HbfError(rc, "hbf_set_head_entries")

    def set_tile_balance(self, on: bool):
        rc = lib().hbf_set_tile_balance(self._h, 1 if on else 0)
        if rc != 0:
            raise HbfError(rc, "hbf_set_tile_balance")

    # ---- thermal ------------------------------------------------------------------------------
    def set_thermal_path(self, generic_only: bool):
        rc = lib().hbf_set_thermal_path(self._h, 1 if generic_only else 0)
        if rc != 0:
            raise HbfError(rc, "hbf_set_thermal_path")

    def thermal_step(self, dt_ns, ext_power_w=None, d_temps_out=None, want_hot=True, check=True):
        hot = np.empty(3, np.float32) if want_hot else None
        if ext_power_w is None:
            p, n = None, 0
        else:
            ext = np.ascontiguousarray(ext_power_w, np.float32)
            p, n = ext.ctypes.data, ext.shape[0]
        rc = lib().hbf_thermal_step(self._h, dt_ns, p, n, _ptr(d_temps_out), hot.ctypes.data if want_hot else None)
        if rc != 0:
            if check:
                raise HbfError(rc, "hbf_thermal_step")
            return rc
        return hot

    def debug_wait_test(self, poll_limit=0, stage=0, tile=0):
        """Test support (``hbf_debug_wait_test``): a small poll budget and one silent tile make the bounded waits run out."""
        rc = lib().hbf_debug_wait_test(self._h, poll_limit, stage, tile)
        if rc != 0:
            raise HbfError(rc, "hbf_debug_wait_test")

    def force_mode(self, mode, q_ppm):
        rc = lib().hbf_force_mode(self._h, mode, q_ppm)
        if rc != 0:
            raise HbfError(rc, "hbf_force_mode")

    def get_mode(self):
        m, q = C.c_int32(), C.c_int64()
        lib().hbf_get_mode(self._h, C.byref(m), C.byref(q))
        return m.value, q.value

    def reset(self):
        rc = lib().hbf_reset(self._h)
        if rc != 0:
            raise HbfError(rc, "hbf_reset")

    # ---- state --------------------------------------------------------------------------------
    def get_busy_until(self):
        out = np.empty(self.n_queues, np.int64)
        rc = lib().hbf_get_busy_until(self._h, out.ctypes.data, out.shape[0])
        if rc != 0:
            raise HbfError(rc, "hbf_get_busy_until")
        return out

    def get_pending_energy(self):
        out = np.empty(self.n_dies, np.int64)
        rc = lib().hbf_get_pending_energy(self._h, out.ctypes.data, out.shape[0])
        if rc != 0:
            raise HbfError(rc, "hbf_get_pending_energy")
        return out

    def get_temps(self):
        out = np.empty(self.n_cells, np.float32)
        rc = lib().hbf_get_temps(self._h, out.ctypes.data, out.shape[0])
        if rc != 0:
            raise HbfError(rc, "hbf_get_temps")
        return out

    def euler_limit_ns(self):
        return lib().hbf_euler_limit_ns(self._h)

    def set_profiling(self, on: bool):
        rc = lib().hbf_set_profiling(self._h, 1 if on else 0)
        if rc != 0:
            raise HbfError(rc, "hbf_set_profiling")

    def get_profile(self) -> dict:
        ms = np.zeros(len(PROF_STAGES), np.float32)
        rc = lib().hbf_get_profile(self._h, ms.ctypes.data, ms.shape[0])
        if rc != 0:
            raise HbfError(rc, "hbf_get_profile")
        return dict(zip(PROF_STAGES, ms.tolist()))

    def get_state(self) -> bytes:
        sz = C.c_size_t()
        lib().hbf_get_state(self._h, None, C.byref(sz))
        buf = C.create_string_buffer(sz.value)
        rc = lib().hbf_get_state(self._h, buf, C.byref(sz))
        if rc != 0:
            raise HbfError(rc, "hbf_get_state")
        return buf.raw[:sz.value]

    def set_state(self, blob: bytes):
        rc = lib().hbf_set_state(self._h, blob, len(blob))
        if rc != 0:
            raise HbfError(rc, "hbf_set_state")

    # ---- host buffers through the library's copy pipeline --------------------------------------------------------
    def submit_pinned(self, h_acc, n, h_completion, h_stall, h_die_stats=None, chunk=0):
        """``hbf_submit_host``: serves a batch that lives in host memory (torch CPU tensors, pinned for overlapped copies:
        h_acc int64 [3 n] (the records), h_completion, h_stall int64 [n], h_die_stats int64 [6 dies] or None).  The
        library cuts it into chunks and overlaps copy-in, service and read-back; the call returns when the results are in
        the caller's buffers.  Returns (code, summary dict)."""
        r = hbf_batch_result_t()
        rc = lib().hbf_submit_host(self._h, _ptr(h_acc), n, _ptr(h_completion), _ptr(h_stall), _ptr(h_die_stats), chunk, C.byref(r))
        return rc, r.as_dict()

    # ---- host-buffer convenience: copies in, one submit, copies out ---------------------------------
    def submit_host(self, acc: np.ndarray, want_status=True, check=True, parts_capacity=None):
        """Marshals a host batch through the device: H2D of the records, ``hbf_submit_batch`` (or, with
        parts_capacity given, ``hbf_submit_batch_paged``), D2H of completions, stalls, status and per-die stats.
        Returns (code, completion, stall, status, die_stats)."""
        torch = self._torch
        acc = np.ascontiguousarray(acc, dtype=ACCESS_DTYPE)
        n = acc.shape[0]
        with torch.cuda.stream(self.stream):
            d_acc = torch.from_numpy(acc.view(np.int64).reshape(-1)).cuda() if n else torch.empty(0, dtype=torch.int64, device="cuda")
            d_comp = torch.empty(n, dtype=torch.int64, device="cuda")
            d_stall = torch.empty(n, dtype=torch.int64, device="cuda")
            d_status = torch.empty(n, dtype=torch.uint8, device="cuda") if want_status else None
            d_ds = torch.empty(self.n_dies * 6, dtype=torch.int64, device="cuda")
            if parts_capacity is None:
                rc = self.submit_batch(d_acc, n, d_comp, d_stall, d_status, d_ds)
            else:
                rc = self.submit_batch_paged(d_acc, n, parts_capacity, d_comp, d_stall, d_status, d_ds)
            if rc != 0:
                if check:
                    raise HbfError(rc, "hbf_submit_batch")
                return rc, None, None, None, None
            res = self.last_result()
            if check and res["code"] != 0:
                raise HbfError(res["code"], "batch")
            comp, stall = d_comp.cpu().numpy(), d_stall.cpu().numpy()
            status = d_status.cpu().numpy() if want_status else None
            ds = d_ds.cpu().numpy().view(DIE_STATS_DTYPE)
        return res["code"], comp, stall, status, ds


class Rom:
    """Reduced-order thermal model (Eq. 2) on the device: ``hbf_rom_create`` / ``hbf_rom_step``."""

    def __init__(self, A, B, C_, D=None, b=None, d=None, stream=None):
        import torch
        self._torch = torch
        A = np.ascontiguousarray(A, np.float64); B = np.ascontiguousarray(B, np.float64); C_ = np.ascontiguousarray(C_, np.float64)
        self.n, self.m, self.o = A.shape[0], B.shape[1], C_.shape[0]
        opt = lambda v, shape: None if v is None else np.ascontiguousarray(np.broadcast_to(np.asarray(v, np.float64), shape))
        D, b, d = opt(D, (self.o, self.m)), opt(b, (self.n,)), opt(d, (self.o,))
        ptr = lambda v: None if v is None else v.ctypes.data
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        h = C.c_void_p()
        rc = lib().hbf_rom_create(self.n, self.m, self.o, ptr(A), ptr(B), ptr(b), ptr(C_), ptr(D), ptr(d),
                                  self.stream.cuda_stream, C.byref(h))
        if rc != 0:
            raise HbfError(rc, "hbf_rom_create")
        self._h = h

    def __del__(self):
        try:
            if getattr(self, "_h", None):
                lib().hbf_rom_destroy(self._h); self._h = None
        except Exception:
            pass

    def reset(self):
        lib().hbf_rom_reset(self._h)

    def step_device(self, d_power, n_steps, d_temps_out):
        rc = lib().hbf_rom_step(self._h, _ptr(d_power), n_steps, _ptr(d_temps_out))
        if rc != 0:
            raise HbfError(rc, "hbf_rom_step")

    def step(self, power):
        """Host convenience: power [n_steps][n_inputs] -> temperatures [n_steps][n_outputs] (copies in and out)."""
        torch = self._torch
        p = np.ascontiguousarray(np.atleast_2d(power), np.float64)
        with torch.cuda.stream(self.stream):
            d_p = torch.from_numpy(p).cuda()
            d_t = torch.empty((p.shape[0], self.o), dtype=torch.float64, device="cuda")
            self.step_device(d_p, p.shape[0], d_t)
            return d_t.cpu().numpy()

    def state(self):
        x = np.empty(self.n, np.float64)
        lib().hbf_rom_get_state(self._h, x.ctypes.data, self.n)
        return x
