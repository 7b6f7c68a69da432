"""Python binding of the B200 HAG aggregation library.

Thin argument marshalling over the C ABI declared in ``include/hag.h``: every
step of the aggregation runs in the library's CUDA kernels.  PyTorch supplies
device memory and streams only.  There is no CPU fallback: if the shared
library is missing the first call raises.

    h = Hag.build(row_ptr, col_idx, capacity)   # Algorithm 3 (host)
    h.to_device(0)
    out = h.aggregate_fwd(x, reduce="mean")     # Algorithm 2
    gx = h.aggregate_bwd(grad_out, reduce="mean")
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhag_b200.so")

HAG_SUM, HAG_MEAN, HAG_GCN = 0, 1, 2
HAG_F32, HAG_BF16 = 0, 1
(HAG_OK, HAG_ERR_NULL, HAG_ERR_ARG, HAG_ERR_GRAPH, HAG_ERR_OOM_HOST, HAG_ERR_OOM_DEVICE, HAG_ERR_CUDA, HAG_ERR_DTYPE,
 HAG_ERR_ALIGN, HAG_ERR_WORKSPACE, HAG_ERR_TIMEOUT, HAG_ERR_NOT_ON_DEVICE, HAG_ERR_TOO_LARGE) = range(13)

EXPORTED_SYMBOLS = [
    "hag_build", "hag_build_ex", "hag_build_threads", "hag_truncate", "hag_import", "hag_export_row_order", "hag_device_validate", "hag_test_range_predicates", "hag_set_cuts", "hag_destroy", "hag_get_info", "hag_export", "hag_to_device", "hag_workspace_bytes", "csr_workspace_bytes",
    "hag_aggregate_fwd", "hag_aggregate_bwd", "csr_aggregate_fwd", "csr_aggregate_bwd",
    "hag_aggregate_host", "hag_aggregate_fwd_static", "hag_graph_pool_fwd", "hag_graph_pool_bwd",
    "hag_max_workspace_bytes", "hag_max_fwd", "hag_max_bwd", "csr_max_fwd", "csr_max_bwd", "hag_profile_enable", "hag_profile_read", "hag_last_launch_count", "hag_status_str",
    "hag_set_schedule", "hag_device_status", "hag_selftest_wait_limit", "hag_export_pass", "hag_test_fail_allocation",
]


class HagError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {status_str(status)} (status {status})")
        self.status = status


class HagInfo(ctypes.Structure):
    _fields_ = [
        ("n", ctypes.c_int32), ("capacity", ctypes.c_int32), ("num_agg", ctypes.c_int32),
        ("num_levels", ctypes.c_int32), ("e", ctypes.c_int64), ("e_hat", ctypes.c_int64),
        ("aggregations_gnn", ctypes.c_int64), ("aggregations_hag", ctypes.c_int64),
        ("aggregations_hag_closed", ctypes.c_int64), ("saved", ctypes.c_int64),
        ("first_redundancy", ctypes.c_int32), ("last_redundancy", ctypes.c_int32),
        ("max_in_degree", ctypes.c_int32), ("max_res_degree", ctypes.c_int32),
        ("max_out_degree", ctypes.c_int32), ("device", ctypes.c_int32),
        ("build_seconds", ctypes.c_double),
    ]

    def as_dict(self) -> dict:
        return {k: getattr(self, k) for k, _ in self._fields_}


class HagPassView(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int64) for k in ("n_rows", "n_phases", "n_chunk_rows", "n_ids")] + [
        (k, ctypes.c_void_p) for k in ("rows", "phase_size", "ids")]


class HagArrays(ctypes.Structure):
    _fields_ = [("n", ctypes.c_int32), ("num_agg", ctypes.c_int32), ("num_levels", ctypes.c_int32)] + [
        (k, ctypes.c_void_p) for k in ("level_ptr", "agg_in", "res_ptr", "res_idx", "t_ptr", "t_idx", "in_degree",
                                       "trace", "csr_t_ptr", "csr_t_idx")] + [
        ("fwd_cut", ctypes.c_int32), ("bwd_cut", ctypes.c_int32)] + [
        (k, ctypes.c_void_p) for k in ("ftail_ptr", "ftail_idx", "btail_ptr", "btail_idx")]


_lib = None


def load_library():
    """Load the shared library (raises if it has not been built)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_1906_03707_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    lib.hag_build.argtypes = [i32, vp, vp, i32, ctypes.POINTER(vp)]
    lib.hag_build.restype = ctypes.c_int
    lib.hag_build_ex.argtypes = [i32, vp, vp, i32, i32, ctypes.POINTER(vp)]
    lib.hag_build_ex.restype = ctypes.c_int
    lib.hag_build_threads.argtypes = [i32]
    lib.hag_build_threads.restype = i32
    lib.hag_truncate.argtypes = [vp, i32, ctypes.POINTER(vp)]
    lib.hag_truncate.restype = ctypes.c_int
    lib.hag_export_row_order.argtypes = [vp, i32, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(vp)]
    lib.hag_export_row_order.restype = ctypes.c_int
    lib.hag_device_validate.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32), vp]
    lib.hag_device_validate.restype = ctypes.c_int
    lib.hag_test_range_predicates.argtypes = [i32, i32, i32, ctypes.c_int64, ctypes.c_int64, i32, i32, i32, i32]
    lib.hag_test_range_predicates.restype = i32
    lib.hag_import.argtypes = [i32, vp, vp, i32, vp, ctypes.POINTER(vp)]
    lib.hag_import.restype = ctypes.c_int
    lib.hag_set_cuts.argtypes = [vp, i32, i32]
    lib.hag_set_cuts.restype = ctypes.c_int
    lib.hag_destroy.argtypes = [vp]
    lib.hag_destroy.restype = ctypes.c_int
    lib.hag_get_info.argtypes = [vp, ctypes.POINTER(HagInfo)]
    lib.hag_get_info.restype = ctypes.c_int
    lib.hag_export.argtypes = [vp, ctypes.POINTER(HagArrays)]
    lib.hag_export.restype = ctypes.c_int
    lib.hag_to_device.argtypes = [vp, ctypes.c_int]
    lib.hag_to_device.restype = ctypes.c_int
    lib.hag_workspace_bytes.argtypes = [vp, i32]
    lib.hag_workspace_bytes.restype = ctypes.c_size_t
    lib.csr_workspace_bytes.argtypes = [vp, i32]
    lib.csr_workspace_bytes.restype = ctypes.c_size_t
    for name in ("hag_aggregate_fwd", "hag_aggregate_bwd", "csr_aggregate_fwd", "csr_aggregate_bwd"):
        f = getattr(lib, name)
        f.argtypes = [vp, ctypes.c_int, ctypes.c_int, i32, vp, vp, vp, vp]
        f.restype = ctypes.c_int
    lib.hag_aggregate_host.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, i32, vp, vp, vp]
    lib.hag_aggregate_host.restype = ctypes.c_int
    lib.hag_aggregate_fwd_static.argtypes = [vp, ctypes.c_int, ctypes.c_int, i32, vp, vp, vp]
    lib.hag_aggregate_fwd_static.restype = ctypes.c_int
    lib.hag_graph_pool_fwd.argtypes = [vp, i32, ctypes.c_int, ctypes.c_int, i32, vp, vp, vp]
    lib.hag_graph_pool_fwd.restype = ctypes.c_int
    lib.hag_graph_pool_bwd.argtypes = [vp, i32, i32, ctypes.c_int, ctypes.c_int, i32, vp, vp, vp]
    lib.hag_graph_pool_bwd.restype = ctypes.c_int
    lib.hag_max_workspace_bytes.argtypes = [vp, i32]
    lib.hag_max_workspace_bytes.restype = ctypes.c_size_t
    lib.hag_max_fwd.argtypes = [vp, ctypes.c_int, i32, vp, vp, vp, vp]
    lib.hag_max_fwd.restype = ctypes.c_int
    lib.hag_max_bwd.argtypes = [vp, ctypes.c_int, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.hag_max_bwd.restype = ctypes.c_int
    lib.csr_max_fwd.argtypes = [vp, ctypes.c_int, i32, vp, vp, vp]
    lib.csr_max_fwd.restype = ctypes.c_int
    lib.csr_max_bwd.argtypes = [vp, ctypes.c_int, i32, vp, vp, vp, vp, vp]
    lib.csr_max_bwd.restype = ctypes.c_int
    lib.hag_profile_enable.argtypes = [vp, ctypes.c_int]
    lib.hag_profile_enable.restype = ctypes.c_int
    lib.hag_profile_read.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.hag_profile_read.restype = i32
    lib.hag_last_launch_count.argtypes = [vp]
    lib.hag_last_launch_count.restype = i32
    lib.hag_set_schedule.argtypes = [vp, i32]
    lib.hag_set_schedule.restype = ctypes.c_int
    lib.hag_device_status.argtypes = [vp]
    lib.hag_device_status.restype = ctypes.c_int
    lib.hag_selftest_wait_limit.argtypes = [vp, vp]
    lib.hag_selftest_wait_limit.restype = ctypes.c_int
    lib.hag_export_pass.argtypes = [vp, i32, ctypes.POINTER(HagPassView)]
    lib.hag_export_pass.restype = ctypes.c_int
    lib.hag_test_fail_allocation.argtypes = [i32, i32]
    lib.hag_test_fail_allocation.restype = ctypes.c_int
    lib.hag_status_str.argtypes = [ctypes.c_int]
    lib.hag_status_str.restype = ctypes.c_char_p
    _lib = lib
    return lib


def build_threads(threads: int = -1) -> int:
    """``hag_build_threads``: set (>= 0) or query (< 0) the host threads of the search; returns the previous value."""
    return int(load_library().hag_build_threads(int(threads)))


def status_str(status: int) -> str:
    return load_library().hag_status_str(int(status)).decode()


def _check(status: int, what: str):
    if status != 0:
        raise HagError(status, what)


def _reduce_code(reduce) -> int:
    if reduce in ("sum", HAG_SUM):
        return HAG_SUM
    if reduce in ("mean", HAG_MEAN):
        return HAG_MEAN
    if reduce in ("gcn", HAG_GCN):
        return HAG_GCN
    raise ValueError(f"reduce must be 'sum', 'mean' or 'gcn', got {reduce!r}")


def _view(ptr, count, dtype):
    if count == 0 or not ptr:
        return np.zeros(0, dtype=dtype)
    ctype = {np.int32: ctypes.c_int32, np.int64: ctypes.c_int64}[dtype]
    return np.ctypeslib.as_array(ctypes.cast(ptr, ctypes.POINTER(ctype)), shape=(count,)).copy()


class Hag:
    """A built HAG: owns the library handle."""

    def __init__(self, handle):
        self._h = handle
        self._ws = None
        self._device = -1
        self._n = int(self.info()["n"])

    # -- construction ------------------------------------------------------- #
    @classmethod
    def build(cls, row_ptr, col_idx, capacity: int, min_redundancy: int = 2) -> "Hag":
        """``hag_build`` / ``hag_build_ex``: CSR of in-neighbours on the host (int64 row_ptr, int32 col_idx)."""
        lib = load_library()
        rp = np.ascontiguousarray(row_ptr, dtype=np.int64)
        ci = np.ascontiguousarray(col_idx, dtype=np.int32)
        handle = ctypes.c_void_p()
        n = rp.shape[0] - 1
        st = lib.hag_build_ex(n, rp.ctypes.data, ci.ctypes.data if ci.size else None, int(capacity),
                              int(min_redundancy), ctypes.byref(handle))
        _check(st, "hag_build")
        return cls(handle)

    @classmethod
    def from_trace(cls, row_ptr, col_idx, trace) -> "Hag":
        """``hag_import``: the HAG of the graph from a recorded merge trace (``arrays()["trace"]``), no search."""
        lib = load_library()
        rp = np.ascontiguousarray(row_ptr, dtype=np.int64)
        ci = np.ascontiguousarray(col_idx, dtype=np.int32)
        tr = np.ascontiguousarray(np.asarray(trace, dtype=np.int32).reshape(-1, 3))
        handle = ctypes.c_void_p()
        st = lib.hag_import(rp.shape[0] - 1, rp.ctypes.data, ci.ctypes.data if ci.size else None, tr.shape[0],
                            tr.ctypes.data if tr.size else None, ctypes.byref(handle))
        _check(st, "hag_import")
        return cls(handle)

    def truncate(self, capacity: int) -> "Hag":
        """``hag_truncate``: the HAG of the same graph for a smaller capacity, from the recorded merges."""
        handle = ctypes.c_void_p()
        _check(load_library().hag_truncate(self._h, int(capacity), ctypes.byref(handle)), "hag_truncate")
        return Hag(handle)

    def set_cuts(self, fwd_cut: int = -1, bwd_cut: int = -1) -> "Hag":
        """``hag_set_cuts``: force the levels evaluated level by level (-1 keeps the library's choice)."""
        _check(load_library().hag_set_cuts(self._h, int(fwd_cut), int(bwd_cut)), "hag_set_cuts")
        return self

    def close(self):
        if self._h:
            load_library().hag_destroy(self._h)
            self._h = None
            self._ws = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- inspection --------------------------------------------------------- #
    def info(self) -> dict:
        out = HagInfo()
        _check(load_library().hag_get_info(self._h, ctypes.byref(out)), "hag_get_info")
        return out.as_dict()

    def arrays(self) -> dict:
        """Copies of the canonical host arrays (``hag_export``)."""
        a = HagArrays()
        _check(load_library().hag_export(self._h, ctypes.byref(a)), "hag_export")
        n, k, lv = a.n, a.num_agg, a.num_levels
        res_ptr = _view(a.res_ptr, n + 1, np.int64)
        t_ptr = _view(a.t_ptr, n + k + 1, np.int64)
        csr_t_ptr = _view(a.csr_t_ptr, n + 1, np.int64)
        level_ptr = _view(a.level_ptr, lv + 1, np.int64)
        ftail_ptr = _view(a.ftail_ptr, k - int(level_ptr[a.fwd_cut]) + 1, np.int64)
        btail_ptr = _view(a.btail_ptr, k - int(level_ptr[a.bwd_cut]) + 1, np.int64)
        return dict(
            fwd_cut=a.fwd_cut, bwd_cut=a.bwd_cut, ftail_ptr=ftail_ptr, btail_ptr=btail_ptr,
            ftail_idx=_view(a.ftail_idx, int(ftail_ptr[-1]), np.int32),
            btail_idx=_view(a.btail_idx, int(btail_ptr[-1]), np.int32),
            n=n, num_agg=k, num_levels=lv,
            level_ptr=_view(a.level_ptr, lv + 1, np.int64),
            agg_in=_view(a.agg_in, 2 * k, np.int32),
            res_ptr=res_ptr, res_idx=_view(a.res_idx, int(res_ptr[-1]) if n >= 0 and res_ptr.size else 0, np.int32),
            t_ptr=t_ptr, t_idx=_view(a.t_idx, int(t_ptr[-1]) if t_ptr.size else 0, np.int32),
            in_degree=_view(a.in_degree, n, np.int32),
            trace=_view(a.trace, 3 * k, np.int32).reshape(-1, 3),
            csr_t_ptr=csr_t_ptr, csr_t_idx=_view(a.csr_t_idx, int(csr_t_ptr[-1]) if csr_t_ptr.size else 0, np.int32),
        )

    def pass_rows(self, which: int) -> dict:
        """``hag_export_pass``: copies of the row list of one pass (0 fwd, 1 bwd, 2 plain fwd, 3 plain bwd)."""
        v = HagPassView()
        _check(load_library().hag_export_pass(self._h, int(which), ctypes.byref(v)), "hag_export_pass")
        return dict(rows=_view(v.rows, 4 * v.n_rows, np.int32).reshape(-1, 4), phase_size=_view(v.phase_size, v.n_phases, np.int32),
                    ids=_view(v.ids, v.n_ids, np.int32), n_chunk_rows=int(v.n_chunk_rows))

    def row_order(self, which: int):
        """``hag_export_row_order``: (first_row, order) of one list; order is empty where rows are taken as they are."""
        first, count, ptr = ctypes.c_int32(), ctypes.c_int64(), ctypes.c_void_p()
        _check(load_library().hag_export_row_order(self._h, int(which), ctypes.byref(first), ctypes.byref(count), ctypes.byref(ptr)),
               "hag_export_row_order")
        order = _view(ptr.value, count.value, np.int32).copy() if count.value else np.zeros(0, np.int32)
        return int(first.value), order

    def set_schedule(self, schedule) -> "Hag":
        """``hag_set_schedule``: 0 / False a launch per level, 1 / True one launch per pass, 2 the aggregation nodes in one
        launch and the graph nodes in a second."""
        _check(load_library().hag_set_schedule(self._h, int(schedule)), "hag_set_schedule")
        return self

    def device_validate(self, stream=None) -> int:
        """``hag_device_validate``: 0 if every uploaded index array passes the device-side range checks, else the mask of
        failed lists (raises for any other error)."""
        mask = ctypes.c_uint32(0)
        st = load_library().hag_device_validate(self._h, ctypes.byref(mask), stream)
        if st not in (0, 3):
            _check(st, "hag_device_validate")
        return int(mask.value)

    def device_status(self) -> int:
        """``hag_device_status``: 0, or HAG_ERR_TIMEOUT if a device-side wait gave up (call after synchronising)."""
        return int(load_library().hag_device_status(self._h))

    def workspace_bytes(self, d: int) -> int:
        return int(load_library().hag_workspace_bytes(self._h, int(d)))

    def csr_workspace_bytes(self, d: int) -> int:
        return int(load_library().csr_workspace_bytes(self._h, int(d)))

    @property
    def last_launch_count(self) -> int:
        return int(load_library().hag_last_launch_count(self._h))

    def profile(self, enable: bool):
        """``hag_profile_enable``: bracket every launch with CUDA events."""
        _check(load_library().hag_profile_enable(self._h, int(bool(enable))), "hag_profile_enable")

    def profile_read(self):
        """``hag_profile_read``: list of (ms, kind, rows, edges) for the launches of the last call."""
        lib = load_library()
        n = lib.hag_profile_read(self._h, 0, None, None, None, None)
        if n < 0:
            raise HagError(6, "hag_profile_read")
        ms = np.zeros(max(n, 1), np.float32)
        kind = np.zeros(max(n, 1), np.int32)
        rows = np.zeros(max(n, 1), np.int64)
        edges = np.zeros(max(n, 1), np.int64)
        got = lib.hag_profile_read(self._h, n, ms.ctypes.data, kind.ctypes.data, rows.ctypes.data, edges.ctypes.data)
        if got < 0:
            raise HagError(6, "hag_profile_read")
        return [(float(ms[i]), int(kind[i]), int(rows[i]), int(edges[i])) for i in range(n)]

    # -- device ------------------------------------------------------------- #
    def to_device(self, device: int = 0) -> "Hag":
        _check(load_library().hag_to_device(self._h, int(device)), "hag_to_device")
        self._device = int(device)
        return self

    def _workspace(self, d: int, device):
        import torch
        need = max(self.workspace_bytes(d), self.csr_workspace_bytes(d))
        if need == 0:
            return None
        if self._ws is None or self._ws.numel() * 4 < need or self._ws.device != device:
            self._ws = torch.empty(need // 4, dtype=torch.float32, device=device)
        return self._ws

    @staticmethod
    def _dtype_code(t) -> int:
        import torch
        if t.dtype == torch.float32:
            return HAG_F32
        if t.dtype == torch.bfloat16:
            return HAG_BF16
        raise TypeError(f"features must be float32 or bfloat16, got {t.dtype}")

    def _matrix(self, t, what, like=None, host=False):
        """The C ABI takes raw pointers and trusts the caller on sizes: every tensor that reaches it is
        checked here (device of the handle, 2-D, contiguous, N rows, dtype), so that a wrong argument is
        a Python error and never an out-of-range device access."""
        import torch
        if not isinstance(t, torch.Tensor) or t.dim() != 2 or not t.is_contiguous():
            raise ValueError(f"{what} must be a contiguous 2-D tensor")
        if t.shape[0] != self._n:
            raise ValueError(f"{what} has {t.shape[0]} rows, the graph has {self._n} nodes")
        if t.shape[1] <= 0:
            raise ValueError(f"{what} has no columns")
        self._dtype_code(t)
        if host:
            if t.is_cuda:
                raise ValueError(f"{what} must be a host tensor")
        else:
            if self._device < 0:
                raise HagError(HAG_ERR_NOT_ON_DEVICE, what)
            if not t.is_cuda or t.device.index != self._device:
                raise ValueError(f"{what} must live on cuda:{self._device}, the handle's device")
        if like is not None and (t.shape != like.shape or t.dtype != like.dtype or t.device != like.device):
            raise ValueError(f"{what} must match the input's shape, dtype and device")
        return t

    def _scratch(self, ws, need_bytes, what="workspace"):
        import torch
        if need_bytes == 0:
            return
        if (not isinstance(ws, torch.Tensor) or not ws.is_cuda or ws.device.index != self._device
                or not ws.is_contiguous() or ws.numel() * ws.element_size() < need_bytes):
            raise ValueError(f"{what} must be a contiguous tensor of at least {need_bytes} bytes on cuda:{self._device}")

    def _run(self, name, use_hag, inp, reduce, out, workspace):
        import torch
        self._matrix(inp, "features")
        if out is None:
            out = torch.empty_like(inp)
        else:
            self._matrix(out, "out", like=inp)
        d = inp.shape[1]
        stream = torch.cuda.current_stream(inp.device).cuda_stream
        lib = load_library()
        code = self._dtype_code(inp)
        ws = workspace if workspace is not None else self._workspace(d, inp.device)
        self._scratch(ws, self.workspace_bytes(d) if use_hag else self.csr_workspace_bytes(d))
        st = getattr(lib, name)(self._h, _reduce_code(reduce), code, d, inp.data_ptr(), out.data_ptr(),
                                ws.data_ptr() if ws is not None else None, stream)
        _check(st, name)
        return out

    def aggregate_fwd(self, x, reduce="sum", out=None, workspace=None):
        """``hag_aggregate_fwd`` on the current stream."""
        return self._run("hag_aggregate_fwd", True, x, reduce, out, workspace)

    def aggregate_bwd(self, grad_out, reduce="sum", out=None, workspace=None):
        """``hag_aggregate_bwd`` on the current stream."""
        return self._run("hag_aggregate_bwd", True, grad_out, reduce, out, workspace)

    def aggregate_fwd_static(self, x, out, reduce="sum"):
        """``hag_aggregate_fwd_static``: the forward pass for hosts that may not allocate
        device memory.  The caller supplies ``out``; the aggregation-node rows go to the
        scratch array built into the library (one per GPU, shared by all calls, so
        keep calls on one stream).  This wrapper allocates nothing either."""
        import torch
        self._matrix(x, "features")
        self._matrix(out, "out", like=x)
        stream = torch.cuda.current_stream(x.device).cuda_stream
        st = load_library().hag_aggregate_fwd_static(self._h, _reduce_code(reduce), self._dtype_code(x), x.shape[1],
                                                     x.data_ptr(), out.data_ptr(), stream)
        _check(st, "hag_aggregate_fwd_static")
        return out

    def csr_fwd(self, x, reduce="sum", out=None, workspace=None):
        """``csr_aggregate_fwd``: the plain GNN-graph, same kernel."""
        return self._run("csr_aggregate_fwd", False, x, reduce, out, workspace)

    def csr_bwd(self, grad_out, reduce="sum", out=None, workspace=None):
        """``csr_aggregate_bwd``."""
        return self._run("csr_aggregate_bwd", False, grad_out, reduce, out, workspace)

    def max_workspace(self, d: int, device):
        """A fresh buffer of ``hag_max_workspace_bytes`` (the forward pass leaves the aggregation nodes' maxima in it)."""
        import torch
        need = max(int(load_library().hag_max_workspace_bytes(self._h, d)), 16)
        return torch.empty(need // 4, dtype=torch.float32, device=device)

    def max_fwd(self, z, out=None, workspace=None, use_hag=True):
        """``hag_max_fwd`` (or ``csr_max_fwd``).  Returns (out, workspace); keep both for ``max_bwd``."""
        import torch
        self._matrix(z, "z")
        if out is None:
            out = torch.empty_like(z)
        else:
            self._matrix(out, "out", like=z)
        s = torch.cuda.current_stream(z.device).cuda_stream
        lib = load_library()
        if use_hag:
            if workspace is None:
                workspace = self.max_workspace(z.shape[1], z.device)
            self._scratch(workspace, int(lib.hag_max_workspace_bytes(self._h, z.shape[1])))
            st = lib.hag_max_fwd(self._h, self._dtype_code(z), z.shape[1], z.data_ptr(), out.data_ptr(), workspace.data_ptr(), s)
        else:
            st = lib.csr_max_fwd(self._h, self._dtype_code(z), z.shape[1], z.data_ptr(), out.data_ptr(), s)
        _check(st, "hag_max_fwd" if use_hag else "csr_max_fwd")
        return out, workspace

    def max_bwd(self, z, fwd_out, fwd_workspace, grad_out, out=None, workspace=None, use_hag=True):
        """``hag_max_bwd`` (or ``csr_max_bwd``): the gradient with respect to z."""
        import torch
        self._matrix(z, "z")
        self._matrix(fwd_out, "fwd_out", like=z)
        self._matrix(grad_out, "grad_out", like=z)
        if out is None:
            out = torch.empty_like(z)
        else:
            self._matrix(out, "out", like=z)
        s = torch.cuda.current_stream(z.device).cuda_stream
        lib = load_library()
        code = self._dtype_code(z)
        if use_hag:
            if workspace is None:
                workspace = self.max_workspace(z.shape[1], z.device)
            need = int(lib.hag_max_workspace_bytes(self._h, z.shape[1]))
            self._scratch(workspace, need)
            self._scratch(fwd_workspace, need, "fwd_workspace")
            st = lib.hag_max_bwd(self._h, code, z.shape[1], z.data_ptr(), fwd_out.data_ptr(), fwd_workspace.data_ptr(),
                                 grad_out.data_ptr(), out.data_ptr(), workspace.data_ptr(), s)
        else:
            st = lib.csr_max_bwd(self._h, code, z.shape[1], z.data_ptr(), fwd_out.data_ptr(), grad_out.data_ptr(), out.data_ptr(), s)
        _check(st, "hag_max_bwd" if use_hag else "csr_max_bwd")
        return out

    def aggregate_host(self, inp, out, reduce="sum", backward=False, use_hag=True, stream=None):
        """``hag_aggregate_host``: host tensors in and out (pinned for async copies);
        enqueues copy-in, aggregation and copy-out on the stream; the caller synchronises."""
        import torch
        self._matrix(inp, "input", host=True)
        self._matrix(out, "out", like=inp, host=True)
        if self._device < 0:
            raise HagError(HAG_ERR_NOT_ON_DEVICE, "aggregate_host")
        s = torch.cuda.current_stream(self._device).cuda_stream if stream is None else stream
        st = load_library().hag_aggregate_host(self._h, int(backward), int(use_hag), _reduce_code(reduce),
                                               self._dtype_code(inp), inp.shape[1], inp.data_ptr(), out.data_ptr(), s)
        _check(st, "hag_aggregate_host")
        return out


def _pool_args(seg_ptr, t):
    import torch
    if not (seg_ptr.is_cuda and seg_ptr.dtype == torch.int32 and seg_ptr.is_contiguous() and seg_ptr.numel() >= 1):
        raise ValueError("seg_ptr must be a contiguous int32 device tensor of n_graphs + 1 offsets")
    if not (t.is_cuda and t.is_contiguous() and t.dim() == 2 and t.device == seg_ptr.device):
        raise ValueError("features must be a contiguous 2-D tensor on seg_ptr's device")
    return seg_ptr.numel() - 1, Hag._dtype_code(t)


def graph_pool_fwd(seg_ptr, x, reduce="mean", out=None):
    """``hag_graph_pool_fwd``: one row per graph of a batch (graph i = rows seg_ptr[i]..seg_ptr[i+1]-1 of x)."""
    import torch
    n_graphs, code = _pool_args(seg_ptr, x)
    if out is None:
        out = torch.empty((n_graphs, x.shape[1]), dtype=x.dtype, device=x.device)
    with torch.cuda.device(x.device):
        st = load_library().hag_graph_pool_fwd(seg_ptr.data_ptr(), n_graphs, _reduce_code(reduce), code, x.shape[1],
                                               x.data_ptr(), out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    _check(st, "hag_graph_pool_fwd")
    return out


def graph_pool_bwd(seg_ptr, grad_out, n_rows: int, reduce="mean", out=None):
    """``hag_graph_pool_bwd``: the gradient of ``graph_pool_fwd`` for an input of n_rows rows."""
    import torch
    n_graphs, code = _pool_args(seg_ptr, grad_out)
    if out is None:
        out = torch.empty((n_rows, grad_out.shape[1]), dtype=grad_out.dtype, device=grad_out.device)
    with torch.cuda.device(grad_out.device):
        st = load_library().hag_graph_pool_bwd(seg_ptr.data_ptr(), n_graphs, n_rows, _reduce_code(reduce), code,
                                               grad_out.shape[1], grad_out.data_ptr(), out.data_ptr(),
                                               torch.cuda.current_stream().cuda_stream)
    _check(st, "hag_graph_pool_bwd")
    return out
