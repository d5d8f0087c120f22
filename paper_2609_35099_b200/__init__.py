"""Python binding of libe3j (the sm_100a fused equivariant convolution).

Argument marshalling only: every function below has the name of the C entry point
it calls (see include/e3j.h) and passes device pointers of torch tensors straight
through.  torch is used for device memory and streams, nothing else; there is no
CPU or PyTorch fallback -- if the compiled library is missing, or a call fails,
an exception is raised.

    plan = e3j_plan_create("128x0e+128x1o", 3, None, 3)
    rowptr, sender_perm, colptr = e3j_graph_prepare(n_nodes, senders, receivers)
    out = e3j_conv_fwd(plan, x, sh, w, senders, receivers, rowptr)
    gx, gsh, gw = e3j_conv_bwd(plan, x, sh, w, senders, receivers, grad_out,
                               rowptr, sender_perm, colptr)
"""
from __future__ import annotations

import ctypes
from pathlib import Path

__all__ = [
    "E3JError", "Plan", "library_path", "e3j_plan_create", "e3j_plan_destroy", "e3j_plan_info",
    "e3j_plan_paths", "e3j_plan_records", "e3j_plan_signature", "e3j_plan_device_status", "e3j_graph_prepare", "e3j_graph_validate",
    "e3j_conv_fwd_workspace_bytes", "e3j_conv_bwd_workspace_bytes", "e3j_conv_fwd", "e3j_conv_fwd_noalloc", "e3j_noalloc_status",
    "e3j_conv_bwd", "e3j_graph_prepare_padded", "e3j_conv_fwd_padded", "e3j_conv_bwd_padded",
    "e3j_conv_bwd_bwd_workspace_bytes", "e3j_conv_bwd_bwd",
    "e3j_radial_weights", "e3j_conv_radial_fwd_workspace_bytes", "e3j_conv_radial_bwd_workspace_bytes",
    "e3j_conv_radial_fwd", "e3j_conv_radial_bwd", "e3j_conv_radial_vec_fwd", "e3j_conv_radial_vec_fwd_workspace_bytes", "e3j_conv_radial_vec_bwd", "e3j_conv_radial_vec_bwd_workspace_bytes",
    "e3j_tp_fwd", "e3j_tp_bwd", "e3j_bwd_schedule_bytes", "e3j_bwd_schedule_build", "e3j_conv_bwd_scheduled", "e3j_harmonics_fwd", "e3j_harmonics_bwd", "e3j_conv_vec_fwd", "e3j_conv_vec_bwd",
    "e3j_conv_vec_fwd_workspace_bytes", "e3j_conv_vec_bwd_workspace_bytes", "e3j_conv_fwd_f64", "e3j_conv_bwd_f64", "e3j_shard_prepare", "e3j_rows_gather", "e3j_rows_add", "e3j_status_string", "e3j_selftest_bounded_wait", "e3j_launch_count", "E3J_PLAN_GENERIC_ONLY",
    "E3J_PLAN_COLLAPSE_OUTPUTS", "E3J_PLAN_RADIAL_MATERIALISE",
]

E3J_PLAN_GENERIC_ONLY = 1
E3J_PLAN_COLLAPSE_OUTPUTS = 2
E3J_PLAN_RADIAL_MATERIALISE = 4
# status codes of include/e3j.h
E3J_OK, E3J_ERR_INVALID_ARG, E3J_ERR_BAD_IRREPS, E3J_ERR_MUL_NOT_UNIFORM = 0, -1, -2, -3
E3J_ERR_UNSUPPORTED, E3J_ERR_WORKSPACE, E3J_ERR_CUDA, E3J_ERR_GRAPH = -4, -5, -6, -7
_LIB_PATH = Path(__file__).resolve().parent / "libe3j.so"
_lib = None


class E3JError(RuntimeError):
    def __init__(self, status: int, where: str):
        lib = _load()
        msg = lib.e3j_status_string(status).decode()
        if status == -6:
            msg += f" (cudaError {lib.e3j_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [status {status}]")
        self.status = status


class _PlanInfo(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("n_channels", "d_in", "d_sh", "n_paths", "d_out", "nnz", "n_pairs", "specialised")]


class _PathInfo(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("in_index", "l1", "p1", "l2", "L", "p", "x_off", "y_off", "out_off")]


def library_path() -> Path:
    return _LIB_PATH


def _load():
    """Loads libe3j.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not _LIB_PATH.exists():
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2609_35099_b200.build` "
            "(nvcc, sm_100a). There is no CPU or PyTorch fallback.")
    lib = ctypes.CDLL(str(_LIB_PATH))
    vp, i64, i32, sz, u32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t, ctypes.c_uint
    lib.e3j_plan_create.argtypes = [ctypes.POINTER(vp), ctypes.c_char_p, i32, ctypes.c_char_p, i32, u32]
    lib.e3j_plan_destroy.argtypes = [vp]
    lib.e3j_plan_info.argtypes = [vp, ctypes.POINTER(_PlanInfo)]
    lib.e3j_plan_paths.argtypes = [vp, ctypes.POINTER(_PathInfo), i32]
    lib.e3j_plan_records.argtypes = [vp, vp, vp, vp, vp, vp, i32]
    lib.e3j_plan_signature.argtypes = [vp]
    lib.e3j_plan_signature.restype = ctypes.c_char_p
    lib.e3j_plan_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32)]
    lib.e3j_plan_device_status.restype = i32
    lib.e3j_graph_prepare.argtypes = [i64, i64, vp, vp, vp, vp, vp, vp]
    lib.e3j_graph_validate.argtypes = [i64, i64, vp, vp, vp, vp]
    lib.e3j_graph_prepare_padded.argtypes = [i64, i64, vp, vp, vp, vp, vp, vp]
    lib.e3j_conv_fwd_workspace_bytes.argtypes = [vp, i64, i64]
    lib.e3j_conv_fwd_workspace_bytes.restype = sz
    lib.e3j_conv_bwd_workspace_bytes.argtypes = [vp, i64, i64]
    lib.e3j_conv_bwd_workspace_bytes.restype = sz
    lib.e3j_conv_fwd.argtypes = [vp, i64, i64] + [vp] * 8 + [sz, vp]
    lib.e3j_conv_bwd.argtypes = [vp, i64, i64] + [vp] * 13 + [sz, vp]
    lib.e3j_conv_fwd_padded.argtypes = [vp, i64, i64] + [vp] * 8 + [sz, vp]
    lib.e3j_conv_bwd_bwd_workspace_bytes.argtypes = [vp, i64, i64]
    lib.e3j_conv_bwd_bwd_workspace_bytes.restype = sz
    lib.e3j_conv_bwd_bwd.argtypes = [vp, i64, i64] + [vp] * 17 + [sz, vp]
    lib.e3j_conv_bwd_padded.argtypes = [vp, i64, i64] + [vp] * 13 + [sz, vp]
    lib.e3j_conv_fwd_noalloc.argtypes = [vp, i64, i64] + [vp] * 7
    lib.e3j_conv_fwd_noalloc.restype = i32
    lib.e3j_noalloc_status.argtypes = [ctypes.POINTER(ctypes.c_int32)]
    lib.e3j_noalloc_status.restype = i32
    lib.e3j_radial_weights.argtypes = [vp, i64, i32] + [vp] * 4
    lib.e3j_radial_weights.restype = i32
    lib.e3j_conv_radial_fwd_workspace_bytes.argtypes = [vp, i64, i64, i32]
    lib.e3j_conv_radial_fwd_workspace_bytes.restype = sz
    lib.e3j_conv_radial_bwd_workspace_bytes.argtypes = [vp, i64, i64, i32]
    lib.e3j_conv_radial_bwd_workspace_bytes.restype = sz
    lib.e3j_conv_radial_fwd.argtypes = [vp, i64, i64, i32] + [vp] * 9 + [sz, vp]
    lib.e3j_conv_radial_fwd.restype = i32
    lib.e3j_conv_radial_vec_fwd_workspace_bytes.argtypes = [vp, i64, i64, i32]
    lib.e3j_conv_radial_vec_fwd_workspace_bytes.restype = sz
    lib.e3j_conv_radial_vec_fwd.argtypes = [vp, i64, i64, i32] + [vp] * 9 + [sz, vp]
    lib.e3j_conv_radial_vec_fwd.restype = i32
    lib.e3j_conv_radial_vec_bwd_workspace_bytes.argtypes = [vp, i64, i64, i32]
    lib.e3j_conv_radial_vec_bwd_workspace_bytes.restype = sz
    lib.e3j_conv_radial_vec_bwd.argtypes = [vp, i64, i64, i32] + [vp] * 15 + [sz, vp]
    lib.e3j_conv_radial_vec_bwd.restype = i32
    lib.e3j_conv_radial_bwd.argtypes = [vp, i64, i64, i32] + [vp] * 15 + [sz, vp]
    lib.e3j_conv_radial_bwd.restype = i32
    lib.e3j_tp_fwd.argtypes = [vp, i64] + [vp] * 5
    lib.e3j_tp_bwd.argtypes = [vp, i64] + [vp] * 8
    lib.e3j_harmonics_fwd.argtypes = [i32, i64, vp, vp, vp]
    lib.e3j_harmonics_fwd.restype = i32
    lib.e3j_harmonics_bwd.argtypes = [i32, i64, vp, vp, vp, vp]
    lib.e3j_harmonics_bwd.restype = i32
    for name in ("e3j_conv_vec_fwd_workspace_bytes", "e3j_conv_vec_bwd_workspace_bytes"):
        getattr(lib, name).argtypes = [vp, i64, i64]
        getattr(lib, name).restype = sz
    lib.e3j_conv_vec_fwd.argtypes = [vp, i64, i64] + [vp] * 8 + [sz, vp]
    lib.e3j_conv_vec_fwd.restype = i32
    lib.e3j_conv_vec_bwd.argtypes = [vp, i64, i64] + [vp] * 13 + [sz, vp]
    lib.e3j_conv_vec_bwd.restype = i32
    lib.e3j_bwd_schedule_bytes.argtypes = [vp, i64, i64]
    lib.e3j_bwd_schedule_bytes.restype = sz
    lib.e3j_bwd_schedule_build.argtypes = [vp, i64, i64, vp, vp, vp, sz, vp]
    lib.e3j_bwd_schedule_build.restype = i32
    lib.e3j_conv_bwd_scheduled.argtypes = [vp, i64, i64] + [vp] * 9 + [sz, vp]
    lib.e3j_conv_bwd_scheduled.restype = i32
    lib.e3j_conv_f64_workspace_bytes.argtypes = [vp, i64, i64]
    lib.e3j_conv_f64_workspace_bytes.restype = sz
    lib.e3j_conv_fwd_f64.argtypes = [vp, i64, i64] + [vp] * 8 + [sz, vp]
    lib.e3j_conv_fwd_f64.restype = i32
    lib.e3j_conv_bwd_f64.argtypes = [vp, i64, i64] + [vp] * 12 + [sz, vp]
    lib.e3j_conv_bwd_f64.restype = i32
    lib.e3j_shard_prepare_workspace_bytes.argtypes = [i64]
    lib.e3j_shard_prepare_workspace_bytes.restype = sz
    lib.e3j_shard_prepare.argtypes = [i64, i64, i32, i32] + [vp] * 7 + [sz, vp]
    lib.e3j_shard_prepare.restype = i32
    lib.e3j_rows_gather.argtypes = [vp, vp, vp, i64, i64, vp]
    lib.e3j_rows_gather.restype = i32
    lib.e3j_rows_add.argtypes = [vp, vp, vp, i64, i64, vp]
    lib.e3j_rows_add.restype = i32
    lib.e3j_selftest_bounded_wait.argtypes = [vp, u32, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
    lib.e3j_selftest_bounded_wait.restype = i32
    lib.e3j_status_string.argtypes = [i32]
    lib.e3j_status_string.restype = ctypes.c_char_p
    lib.e3j_last_cuda_error.restype = i32
    lib.e3j_launch_count.restype = i64
    for name in ("e3j_plan_create", "e3j_plan_destroy", "e3j_plan_info", "e3j_plan_paths", "e3j_plan_records",
                 "e3j_graph_prepare", "e3j_graph_validate", "e3j_conv_fwd", "e3j_conv_bwd", "e3j_tp_fwd",
                 "e3j_tp_bwd"):
        getattr(lib, name).restype = i32
    _lib = lib
    return lib


def _check(status: int, where: str) -> int:
    if status < 0:
        raise E3JError(status, where)
    return status


class Plan:
    """Owner of one e3j_plan handle (released when the object is collected)."""

    def __init__(self, handle: int):
        self.handle = ctypes.c_void_p(handle)
        info = _PlanInfo()
        _check(_load().e3j_plan_info(self.handle, ctypes.byref(info)), "e3j_plan_info")
        for name, _ in _PlanInfo._fields_:
            setattr(self, name, getattr(info, name))

    def __del__(self):
        try:
            e3j_plan_destroy(self)
        except Exception:
            pass


def e3j_plan_create(irreps_in: str, sh_lmax: int, irreps_out: str | None = None, out_lmax: int = -1,
                    flags: int = 0) -> Plan:
    h = ctypes.c_void_p()
    out = irreps_out.encode() if irreps_out is not None else None
    _check(_load().e3j_plan_create(ctypes.byref(h), irreps_in.encode(), sh_lmax, out, out_lmax, flags),
           "e3j_plan_create")
    return Plan(h.value)


def e3j_plan_destroy(plan: Plan) -> None:
    if plan.handle is not None and plan.handle.value:
        _load().e3j_plan_destroy(plan.handle)
        plan.handle = ctypes.c_void_p()


def e3j_plan_info(plan: Plan) -> dict:
    return {name: getattr(plan, name) for name, _ in _PlanInfo._fields_}


def e3j_plan_signature(plan: Plan) -> str:
    return _load().e3j_plan_signature(plan.handle).decode()


def e3j_plan_device_status(plan: Plan) -> int:
    """Sticky device status of the plan on the current device (0 = fine); synchronises."""
    st = ctypes.c_int32(0)
    _check(_load().e3j_plan_device_status(plan.handle, ctypes.byref(st)), "e3j_plan_device_status")
    return int(st.value)


def e3j_plan_paths(plan: Plan) -> list[dict]:
    arr = (_PathInfo * plan.n_paths)()
    _check(_load().e3j_plan_paths(plan.handle, arr, plan.n_paths), "e3j_plan_paths")
    return [{name: getattr(p, name) for name, _ in _PathInfo._fields_} for p in arr]


def e3j_plan_records(plan: Plan):
    """(i0, i1, i2, i3, val) numpy arrays of the coefficient records (host side)."""
    import numpy as np
    n = plan.nnz
    idx = [np.zeros(n, dtype=np.int32) for _ in range(4)]
    val = np.zeros(n, dtype=np.float64)
    ptr = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    _check(_load().e3j_plan_records(plan.handle, *map(ptr, idx), ptr(val), n), "e3j_plan_records")
    return (*idx, val)


# ----------------------------------------------------------------- marshalling
def _torch():
    import torch
    return torch


def _dev_ptr(t, dtype, shape, name):
    torch = _torch()
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name} must be contiguous {dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} has shape {tuple(t.shape)}, expected {tuple(shape)}")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    torch = _torch()
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _workspace(nbytes: int, like, workspace):
    torch = _torch()
    if workspace is None:
        workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=like.device)
    if workspace.dtype != torch.uint8 or not workspace.is_cuda or workspace.numel() < nbytes:
        raise ValueError("workspace must be a CUDA uint8 tensor of sufficient size")
    return workspace


def e3j_graph_prepare(n_nodes: int, senders, receivers, want_transpose: bool = True, stream=None,
                      _entry: str = "e3j_graph_prepare"):
    """(rowptr, sender_perm, colptr) int32 CUDA tensors; the last two are None unless want_transpose."""
    torch = _torch()
    e = senders.numel()
    rowptr = torch.empty(n_nodes + 1, dtype=torch.int32, device=senders.device)
    perm = torch.empty(max(e, 1), dtype=torch.int32, device=senders.device) if want_transpose else None
    colptr = torch.empty(n_nodes + 1, dtype=torch.int32, device=senders.device) if want_transpose else None
    _check(getattr(_load(), _entry)(n_nodes, e, _dev_ptr(senders, torch.int32, (e,), "senders"),
                                    _dev_ptr(receivers, torch.int32, (e,), "receivers"),
                                    _dev_ptr(rowptr, torch.int32, None, "rowptr"),
                                    _dev_ptr(perm, torch.int32, None, "sender_perm"),
                                    _dev_ptr(colptr, torch.int32, None, "colptr"), _stream(stream)),
           _entry)
    if perm is not None:
        perm = perm[:e]
    return rowptr, perm, colptr


def e3j_graph_prepare_padded(n_nodes: int, senders, receivers, want_transpose: bool = True, stream=None):
    """As e3j_graph_prepare for a padded edge list (edges with receiver >= n_nodes are padding and come last):
    rowptr[n_nodes] is the number of real edges, of sender_perm only that many entries are written."""
    return e3j_graph_prepare(n_nodes, senders, receivers, want_transpose, stream, "e3j_graph_prepare_padded")


def e3j_graph_validate(n_nodes: int, senders, receivers, stream=None) -> int:
    """0 if the graph is usable, else the (negative) E3J_ERR_GRAPH status.  Synchronises."""
    torch = _torch()
    e = senders.numel()
    status = torch.zeros(1, dtype=torch.int32, device=senders.device)
    _check(_load().e3j_graph_validate(n_nodes, e, _dev_ptr(senders, torch.int32, (e,), "senders"),
                                      _dev_ptr(receivers, torch.int32, (e,), "receivers"),
                                      _dev_ptr(status, torch.int32, None, "status"), _stream(stream)),
           "e3j_graph_validate")
    return int(status.item())


def e3j_conv_fwd_workspace_bytes(plan: Plan, n_nodes: int, n_edges: int) -> int:
    return int(_load().e3j_conv_fwd_workspace_bytes(plan.handle, n_nodes, n_edges))


def e3j_conv_bwd_workspace_bytes(plan: Plan, n_nodes: int, n_edges: int) -> int:
    return int(_load().e3j_conv_bwd_workspace_bytes(plan.handle, n_nodes, n_edges))


def e3j_conv_fwd(plan: Plan, x, sh, w, senders, receivers, rowptr=None, out=None, workspace=None,
                 stream=None, _entry: str = "e3j_conv_fwd"):
    torch = _torch()
    n, e = x.shape[0], senders.numel()
    f32, i32 = torch.float32, torch.int32
    if out is None:
        out = torch.empty((n, plan.d_out, plan.n_channels), dtype=f32, device=x.device)
    nbytes = e3j_conv_fwd_workspace_bytes(plan, n, e)
    workspace = _workspace(nbytes, x, workspace)
    _check(getattr(_load(), _entry)(
        plan.handle, n, e,
        _dev_ptr(x, f32, (n, plan.d_in, plan.n_channels), "x"),
        _dev_ptr(sh, f32, (e, plan.d_sh), "sh"),
        _dev_ptr(w, f32, (e, plan.n_paths, plan.n_channels), "w"),
        _dev_ptr(senders, i32, (e,), "senders"), _dev_ptr(receivers, i32, (e,), "receivers"),
        _dev_ptr(rowptr, i32, (n + 1,), "rowptr"),
        _dev_ptr(out, f32, (n, plan.d_out, plan.n_channels), "out"),
        ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)), _entry)
    return out


def e3j_conv_fwd_padded(plan: Plan, x, sh, w, senders, receivers, rowptr, out=None, workspace=None, stream=None):
    """Forward convolution over a padded edge list; rowptr (from e3j_graph_prepare_padded) is required."""
    return e3j_conv_fwd(plan, x, sh, w, senders, receivers, rowptr, out, workspace, stream, "e3j_conv_fwd_padded")


def e3j_conv_fwd_noalloc(plan: Plan, x, sh, w, senders, receivers, out, stream=None):
    """Forward convolution through the allocation-free entry point.

    For callers that must not allocate device memory at call time (engines that reserve everything at
    start-up, plug-ins without an allocator): the kernel's scratch lives inside the library, and this
    wrapper allocates nothing either, so `out` must be passed in.  Calls on one device share that scratch and
    must not overlap on the GPU."""
    torch = _torch()
    n, e = x.shape[0], senders.numel()
    f32, i32 = torch.float32, torch.int32
    _check(_load().e3j_conv_fwd_noalloc(
        plan.handle, n, e,
        _dev_ptr(x, f32, (n, plan.d_in, plan.n_channels), "x"),
        _dev_ptr(sh, f32, (e, plan.d_sh), "sh"),
        _dev_ptr(w, f32, (e, plan.n_paths, plan.n_channels), "w"),
        _dev_ptr(senders, i32, (e,), "senders"), _dev_ptr(receivers, i32, (e,), "receivers"),
        _dev_ptr(out, f32, (n, plan.d_out, plan.n_channels), "out"), _stream(stream)), "e3j_conv_fwd_noalloc")
    return out


def e3j_noalloc_status() -> int:
    """Status word of the allocation-free entry point on the current device (0 = fine; non-zero: a bounded wait
    inside its kernel gave up and the output of that call is invalid).  Reads and clears; synchronises."""
    st = ctypes.c_int32(0)
    _check(_load().e3j_noalloc_status(ctypes.byref(st)), "e3j_noalloc_status")
    return int(st.value)


def e3j_conv_bwd(plan: Plan, x, sh, w, senders, receivers, grad_out, rowptr=None, sender_perm=None,
                 colptr=None, grad_x=True, grad_sh=True, grad_w=True, workspace=None, stream=None,
                 _entry: str = "e3j_conv_bwd"):
    """Returns (grad_x, grad_sh, grad_w).  Each grad_* argument is True (allocate), False/None
    (not wanted) or a preallocated tensor."""
    torch = _torch()
    n, e = x.shape[0], senders.numel()
    f32, i32 = torch.float32, torch.int32

    def alloc(flag, shape):
        if flag is True:
            return torch.empty(shape, dtype=f32, device=x.device)
        return flag if isinstance(flag, torch.Tensor) else None

    grad_x = alloc(grad_x, (n, plan.d_in, plan.n_channels))
    grad_sh = alloc(grad_sh, (e, plan.d_sh))
    grad_w = alloc(grad_w, (e, plan.n_paths, plan.n_channels))
    nbytes = e3j_conv_bwd_workspace_bytes(plan, n, e)
    workspace = _workspace(nbytes, x, workspace)
    _check(getattr(_load(), _entry)(
        plan.handle, n, e,
        _dev_ptr(x, f32, (n, plan.d_in, plan.n_channels), "x"),
        _dev_ptr(sh, f32, (e, plan.d_sh), "sh"),
        _dev_ptr(w, f32, (e, plan.n_paths, plan.n_channels), "w"),
        _dev_ptr(senders, i32, (e,), "senders"), _dev_ptr(receivers, i32, (e,), "receivers"),
        _dev_ptr(rowptr, i32, (n + 1,), "rowptr"),
        _dev_ptr(sender_perm, i32, (e,), "sender_perm"), _dev_ptr(colptr, i32, (n + 1,), "colptr"),
        _dev_ptr(grad_out, f32, (n, plan.d_out, plan.n_channels), "grad_out"),
        _dev_ptr(grad_x, f32, (n, plan.d_in, plan.n_channels), "grad_x"),
        _dev_ptr(grad_sh, f32, (e, plan.d_sh), "grad_sh"),
        _dev_ptr(grad_w, f32, (e, plan.n_paths, plan.n_channels), "grad_w"),
        ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)), _entry)
    return grad_x, grad_sh, grad_w


def e3j_conv_bwd_padded(plan: Plan, x, sh, w, senders, receivers, grad_out, rowptr, sender_perm=None,
                        colptr=None, grad_x=True, grad_sh=True, grad_w=True, workspace=None, stream=None):
    """Backward convolution over a padded edge list; rowptr (from e3j_graph_prepare_padded) is required.
    The grad_sh / grad_w rows of padding edges come back as zeros."""
    return e3j_conv_bwd(plan, x, sh, w, senders, receivers, grad_out, rowptr, sender_perm, colptr, grad_x,
                        grad_sh, grad_w, workspace, stream, "e3j_conv_bwd_padded")


def e3j_conv_bwd_bwd_workspace_bytes(plan: Plan, n_nodes: int, n_edges: int) -> int:
    return int(_load().e3j_conv_bwd_bwd_workspace_bytes(plan.handle, n_nodes, n_edges))


def e3j_conv_bwd_bwd(plan: Plan, x, sh, w, senders, receivers, grad_out, rowptr, sender_perm, colptr,
                     ct_x=None, ct_sh=None, ct_w=None, gg_out=True, g_x=True, g_sh=True, g_w=True,
                     workspace=None, stream=None):
    """Double backward: cotangents (ct_x, ct_sh, ct_w) of the backward's results -> cotangents
    (gg_out, g_x, g_sh, g_w) of the backward's inputs (grad_out, x, sh, w).  A missing ct_* is zero; each
    output argument is True (allocate), False/None (not wanted) or a preallocated tensor."""
    torch = _torch()
    n, e = x.shape[0], senders.numel()
    f32, i32 = torch.float32, torch.int32

    def alloc(flag, shape):
        if flag is True:
            return torch.empty(shape, dtype=f32, device=x.device)
        return flag if isinstance(flag, torch.Tensor) else None

    s_x, s_sh = (n, plan.d_in, plan.n_channels), (e, plan.d_sh)
    s_w, s_out = (e, plan.n_paths, plan.n_channels), (n, plan.d_out, plan.n_channels)
    gg_out, g_x, g_sh, g_w = alloc(gg_out, s_out), alloc(g_x, s_x), alloc(g_sh, s_sh), alloc(g_w, s_w)
    workspace = _workspace(e3j_conv_bwd_bwd_workspace_bytes(plan, n, e), x, workspace)
    _check(_load().e3j_conv_bwd_bwd(
        plan.handle, n, e, _dev_ptr(x, f32, s_x, "x"), _dev_ptr(sh, f32, s_sh, "sh"), _dev_ptr(w, f32, s_w, "w"),
        _dev_ptr(senders, i32, (e,), "senders"), _dev_ptr(receivers, i32, (e,), "receivers"),
        _dev_ptr(rowptr, i32, (n + 1,), "rowptr"), _dev_ptr(sender_perm, i32, (e,), "sender_perm"),
        _dev_ptr(colptr, i32, (n + 1,), "colptr"), _dev_ptr(grad_out, f32, s_out, "grad_out"),
        _dev_ptr(ct_x, f32, s_x, "ct_x"), _dev_ptr(ct_sh, f32, s_sh, "ct_sh"), _dev_ptr(ct_w, f32, s_w, "ct_w"),
        _dev_ptr(gg_out, f32, s_out, "gg_out"), _dev_ptr(g_x, f32, s_x, "g_x"), _dev_ptr(g_sh, f32, s_sh, "g_sh"),
        _dev_ptr(g_w, f32, s_w, "g_w"),
        ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)), "e3j_conv_bwd_bwd")
    return gg_out, g_x, g_sh, g_w


def e3j_radial_weights(plan: Plan, h, W, out=None, stream=None):
    """w[E, P, N_q] = h W (the radial network's last layer), materialised."""
    torch = _torch()
    e, hidden = h.shape
    f32 = torch.float32
    if out is None:
        out = torch.empty((e, plan.n_paths, plan.n_channels), dtype=f32, device=h.device)
    _check(_load().e3j_radial_weights(
        plan.handle, e, hidden, _dev_ptr(h, f32, (e, hidden), "h"),
        _dev_ptr(W, f32, (hidden, plan.n_paths * plan.n_channels), "W"),
        _dev_ptr(out, f32, (e, plan.n_paths, plan.n_channels), "out"), _stream(stream)), "e3j_radial_weights")
    return out


def e3j_conv_radial_fwd_workspace_bytes(plan: Plan, n_nodes: int, n_edges: int, hidden: int) -> int:
    return int(_load().e3j_conv_radial_fwd_workspace_bytes(plan.handle, n_nodes, n_edges, hidden))


def e3j_conv_radial_bwd_workspace_bytes(plan: Plan, n_nodes: int, n_edges: int, hidden: int) -> int:
    return int(_load().e3j_conv_radial_bwd_workspace_bytes(plan.handle, n_nodes, n_edges, hidden))


def e3j_conv_radial_fwd(plan: Plan, x, sh, h, W, senders, receivers, rowptr=None, out=None, workspace=None,
                        stream=None):
    """Forward convolution with the edge weights given as (h [E, hidden], W [hidden, P * N_q])."""
    torch = _torch()
    n, e, hidden = x.shape[0], senders.numel(), W.shape[0]
    f32, i32 = torch.float32, torch.int32
    if out is None:
        out = torch.empty((n, plan.d_out, plan.n_channels), dtype=f32, device=x.device)
    workspace = _workspace(e3j_conv_radial_fwd_workspace_bytes(plan, n, e, hidden), x, workspace)
    _check(_load().e3j_conv_radial_fwd(
        plan.handle, n, e, hidden,
        _dev_ptr(x, f32, (n, plan.d_in, plan.n_channels), "x"), _dev_ptr(sh, f32, (e, plan.d_sh), "sh"),
        _dev_ptr(h, f32, (e, hidden), "h"), _dev_ptr(W, f32, (hidden, plan.n_paths * plan.n_channels), "W"),
        _dev_ptr(senders, i32, (e,), "senders"), _dev_ptr(receivers, i32, (e,), "receivers"),
        _dev_ptr(rowptr, i32, (n + 1,), "rowptr"),
        _dev_ptr(out, f32, (n, plan.d_out, plan.n_channels), "out"),
        ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)), "e3j_conv_radial_fwd")
    return out


def e3j_conv_radial_vec_fwd_workspace_bytes(plan: Plan, n_nodes: int, n_edges: int, hidden: int) -> int:
    return int(_load().e3j_conv_radial_vec_fwd_workspace_bytes(plan.handle, n_nodes, n_edges, hidden))


def e3j_conv_radial_vec_fwd(plan: Plan, x, edge_vec, h, W, senders, receivers, rowptr=None, out=None, workspace=None,
                            stream=None):
    """Forward convolution from edge vectors [E, 3] and the radial layer (h, W): neither the harmonics nor the
    edge weights exist as arrays where the plan has the kernel for it."""
    torch = _torch()
    n, e, hidden = x.shape[0], senders.numel(), W.shape[0]
    f32, i32 = torch.float32, torch.int32
    if out is None:
        out = torch.empty((n, plan.d_out, plan.n_channels), dtype=f32, device=x.device)
    workspace = _workspace(e3j_conv_radial_vec_fwd_workspace_bytes(plan, n, e, hidden), x, workspace)
    _check(_load().e3j_conv_radial_vec_fwd(
        plan.handle, n, e, hidden,
        _dev_ptr(x, f32, (n, plan.d_in, plan.n_channels), "x"), _dev_ptr(edge_vec, f32, (e, 3), "edge_vec"),
        _dev_ptr(h, f32, (e, hidden), "h"), _dev_ptr(W, f32, (hidden, plan.n_paths * plan.n_channels), "W"),
        _dev_ptr(senders, i32, (e,), "senders"), _dev_ptr(receivers, i32, (e,), "receivers"),
        _dev_ptr(rowptr, i32, (n + 1,), "rowptr"),
        _dev_ptr(out, f32, (n, plan.d_out, plan.n_channels), "out"),
        ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)), "e3j_conv_radial_vec_fwd")
    return out


def e3j_conv_radial_bwd(plan: Plan, x, sh, h, W, senders, receivers, grad_out, rowptr=None, sender_perm=None,
                        colptr=None, grad_x=True, grad_sh=True, grad_h=True, grad_W=True, workspace=None,
                        stream=None):
    """Returns (grad_x, grad_sh, grad_h, grad_W); each grad_* argument is True (allocate), False/None (not
    wanted) or a preallocated tensor."""
    torch = _torch()
    n, e, hidden = x.shape[0], senders.numel(), W.shape[0]
    f32, i32 = torch.float32, torch.int32

    def alloc(flag, shape):
        if flag is True:
            return torch.empty(shape, dtype=f32, device=x.device)
        return flag if isinstance(flag, torch.Tensor) else None

    s_w = (hidden, plan.n_paths * plan.n_channels)
    grad_x = alloc(grad_x, (n, plan.d_in, plan.n_channels))
    grad_sh = alloc(grad_sh, (e, plan.d_sh))
    grad_h = alloc(grad_h, (e, hidden))
    grad_W = alloc(grad_W, s_w)
    workspace = _workspace(e3j_conv_radial_bwd_workspace_bytes(plan, n, e, hidden), x, workspace)
    _check(_load().e3j_conv_radial_bwd(
        plan.handle, n, e, hidden,
        _dev_ptr(x, f32, (n, plan.d_in, plan.n_channels), "x"), _dev_ptr(sh, f32, (e, plan.d_sh), "sh"),
        _dev_ptr(h, f32, (e, hidden), "h"), _dev_ptr(W, f32, s_w, "W"),
        _dev_ptr(senders, i32, (e,), "senders"), _dev_ptr(receivers, i32, (e,), "receivers"),
        _dev_ptr(rowptr, i32, (n + 1,), "rowptr"),
        _dev_ptr(sender_perm, i32, (e,), "sender_perm"), _dev_ptr(colptr, i32, (n + 1,), "colptr"),
        _dev_ptr(grad_out, f32, (n, plan.d_out, plan.n_channels), "grad_out"),
        _dev_ptr(grad_x, f32, (n, plan.d_in, plan.n_channels), "grad_x"),
        _dev_ptr(grad_sh, f32, (e, plan.d_sh), "grad_sh"),
        _dev_ptr(grad_h, f32, (e, hidden), "grad_h"), _dev_ptr(grad_W, f32, s_w, "grad_W"),
        ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)), "e3j_conv_radial_bwd")
    return grad_x, grad_sh, grad_h, grad_W


def e3j_conv_radial_vec_bwd_workspace_bytes(plan: Plan, n_nodes: int, n_edges: int, hidden: int) -> int:
    return int(_load().e3j_conv_radial_vec_bwd_workspace_bytes(plan.handle, n_nodes, n_edges, hidden))


def e3j_conv_radial_vec_bwd(plan: Plan, x, edge_vec, h, W, senders, receivers, grad_out, rowptr=None, sender_perm=None,
                            colptr=None, grad_x=True, grad_vec=True, grad_h=True, grad_W=True, workspace=None,
                            stream=None):
    """Backward of e3j_conv_radial_vec_fwd: (grad_x, grad_vec, grad_h, grad_W); each grad_* argument is True
    (allocate), False/None (not wanted) or a preallocated tensor."""
    torch = _torch()
    n, e, hidden = x.shape[0], senders.numel(), W.shape[0]
    f32, i32 = torch.float32, torch.int32

    def alloc(flag, shape):
        if flag is True:
            return torch.empty(shape, dtype=f32, device=x.device)
        return flag if isinstance(flag, torch.Tensor) else None

    s_w = (hidden, plan.n_paths * plan.n_channels)
    grad_x = alloc(grad_x, (n, plan.d_in, plan.n_channels))
    grad_vec = alloc(grad_vec, (e, 3))
    grad_h = alloc(grad_h, (e, hidden))
    grad_W = alloc(grad_W, s_w)
    workspace = _workspace(e3j_conv_radial_vec_bwd_workspace_bytes(plan, n, e, hidden), x, workspace)
    _check(_load().e3j_conv_radial_vec_bwd(
        plan.handle, n, e, hidden,
        _dev_ptr(x, f32, (n, plan.d_in, plan.n_channels), "x"), _dev_ptr(edge_vec, f32, (e, 3), "edge_vec"),
        _dev_ptr(h, f32, (e, hidden), "h"), _dev_ptr(W, f32, s_w, "W"),
        _dev_ptr(senders, i32, (e,), "senders"), _dev_ptr(receivers, i32, (e,), "receivers"),
        _dev_ptr(rowptr, i32, (n + 1,), "rowptr"),
        _dev_ptr(sender_perm, i32, (e,), "sender_perm"), _dev_ptr(colptr, i32, (n + 1,), "colptr"),
        _dev_ptr(grad_out, f32, (n, plan.d_out, plan.n_channels), "grad_out"),
        _dev_ptr(grad_x, f32, (n, plan.d_in, plan.n_channels), "grad_x"), _dev_ptr(grad_vec, f32, (e, 3), "grad_vec"),
        _dev_ptr(grad_h, f32, (e, hidden), "grad_h"), _dev_ptr(grad_W, f32, s_w, "grad_W"),
        ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)), "e3j_conv_radial_vec_bwd")
    return grad_x, grad_vec, grad_h, grad_W


def e3j_tp_fwd(plan: Plan, x1, x2, w, out=None, stream=None):
    torch = _torch()
    rows, f32 = x1.shape[0], torch.float32
    if out is None:
        out = torch.empty((rows, plan.d_out, plan.n_channels), dtype=f32, device=x1.device)
    _check(_load().e3j_tp_fwd(
        plan.handle, rows, _dev_ptr(x1, f32, (rows, plan.d_in, plan.n_channels), "x1"),
        _dev_ptr(x2, f32, (rows, plan.d_sh), "x2"),
        _dev_ptr(w, f32, (rows, plan.n_paths, plan.n_channels), "w"),
        _dev_ptr(out, f32, (rows, plan.d_out, plan.n_channels), "out"), _stream(stream)), "e3j_tp_fwd")
    return out


def e3j_tp_bwd(plan: Plan, x1, x2, w, grad_out, grad_x1=True, grad_x2=True, grad_w=True, stream=None):
    torch = _torch()
    rows, f32 = x1.shape[0], torch.float32

    def alloc(flag, shape):
        if flag is True:
            return torch.empty(shape, dtype=f32, device=x1.device)
        return flag if isinstance(flag, torch.Tensor) else None

    grad_x1 = alloc(grad_x1, (rows, plan.d_in, plan.n_channels))
    grad_x2 = alloc(grad_x2, (rows, plan.d_sh))
    grad_w = alloc(grad_w, (rows, plan.n_paths, plan.n_channels))
    _check(_load().e3j_tp_bwd(
        plan.handle, rows, _dev_ptr(x1, f32, (rows, plan.d_in, plan.n_channels), "x1"),
        _dev_ptr(x2, f32, (rows, plan.d_sh), "x2"),
        _dev_ptr(w, f32, (rows, plan.n_paths, plan.n_channels), "w"),
        _dev_ptr(grad_out, f32, (rows, plan.d_out, plan.n_channels), "grad_out"),
        _dev_ptr(grad_x1, f32, None, "grad_x1"), _dev_ptr(grad_x2, f32, None, "grad_x2"),
        _dev_ptr(grad_w, f32, None, "grad_w"), _stream(stream)), "e3j_tp_bwd")
    return grad_x1, grad_x2, grad_w


def e3j_bwd_schedule_bytes(plan: Plan, n_nodes: int, n_edges: int) -> int:
    """Device bytes a backward schedule may need; 0 if the plan has no scheduled kernel."""
    return int(_load().e3j_bwd_schedule_bytes(plan.handle, n_nodes, n_edges))


def e3j_bwd_schedule_build(plan: Plan, n_nodes: int, senders, receivers, stream=None):
    """The processing order of e3j_conv_bwd_scheduled for this graph (a device uint8 tensor).  The graph arrays may
    live on the device or the host; the order is computed on the host."""
    torch = _torch()
    e = senders.numel()
    dev = senders.device if senders.is_cuda else torch.device("cuda", torch.cuda.current_device())
    nbytes = e3j_bwd_schedule_bytes(plan, n_nodes, e)
    if nbytes == 0:
        raise RuntimeError("e3j_bwd_schedule_build: the plan has no scheduled backward kernel")
    snd = senders.detach().to("cpu", torch.int32).contiguous()
    rcv = receivers.detach().to("cpu", torch.int32).contiguous()
    sched = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    with torch.cuda.device(dev):
        _check(_load().e3j_bwd_schedule_build(plan.handle, n_nodes, e, ctypes.c_void_p(snd.data_ptr()),
                                              ctypes.c_void_p(rcv.data_ptr()), ctypes.c_void_p(sched.data_ptr()), nbytes,
                                              _stream(stream)), "e3j_bwd_schedule_build")
    return sched


def e3j_conv_bwd_scheduled(plan: Plan, x, sh, w, schedule, grad_out, grad_x=None, grad_sh=None, grad_w=None,
                           workspace=None, stream=None):
    """e3j_conv_bwd over a schedule from e3j_bwd_schedule_build: (grad_x, grad_sh, grad_w), all three always."""
    torch = _torch()
    n, e = x.shape[0], w.shape[0]
    f32 = torch.float32
    if grad_x is None:
        grad_x = torch.empty((n, plan.d_in, plan.n_channels), dtype=f32, device=x.device)
    if grad_sh is None:
        grad_sh = torch.empty((e, plan.d_sh), dtype=f32, device=x.device)
    if grad_w is None:
        grad_w = torch.empty((e, plan.n_paths, plan.n_channels), dtype=f32, device=x.device)
    workspace = _workspace(e3j_conv_bwd_workspace_bytes(plan, n, e), x, workspace)
    if schedule.dtype != torch.uint8 or not schedule.is_cuda:
        raise ValueError("schedule must be the CUDA uint8 tensor returned by e3j_bwd_schedule_build")
    _check(_load().e3j_conv_bwd_scheduled(
        plan.handle, n, e, _dev_ptr(x, f32, (n, plan.d_in, plan.n_channels), "x"), _dev_ptr(sh, f32, (e, plan.d_sh), "sh"),
        _dev_ptr(w, f32, (e, plan.n_paths, plan.n_channels), "w"), ctypes.c_void_p(schedule.data_ptr()),
        _dev_ptr(grad_out, f32, (n, plan.d_out, plan.n_channels), "grad_out"),
        _dev_ptr(grad_x, f32, (n, plan.d_in, plan.n_channels), "grad_x"), _dev_ptr(grad_sh, f32, (e, plan.d_sh), "grad_sh"),
        _dev_ptr(grad_w, f32, (e, plan.n_paths, plan.n_channels), "grad_w"),
        ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)), "e3j_conv_bwd_scheduled")
    return grad_x, grad_sh, grad_w


def e3j_harmonics_fwd(lmax: int, edge_vec, out=None, stream=None):
    """sh[E, (lmax+1)^2] = Y(edge_vec / |edge_vec|), component-normalised real harmonics."""
    torch = _torch()
    e, f32 = edge_vec.shape[0], torch.float32
    if out is None:
        out = torch.empty((e, (lmax + 1) ** 2), dtype=f32, device=edge_vec.device)
    _check(_load().e3j_harmonics_fwd(lmax, e, _dev_ptr(edge_vec, f32, (e, 3), "edge_vec"),
                                     _dev_ptr(out, f32, (e, (lmax + 1) ** 2), "sh"), _stream(stream)), "e3j_harmonics_fwd")
    return out


def e3j_harmonics_bwd(lmax: int, edge_vec, grad_sh, out=None, stream=None):
    """grad_vec[E, 3] of e3j_harmonics_fwd."""
    torch = _torch()
    e, f32 = edge_vec.shape[0], torch.float32
    if out is None:
        out = torch.empty((e, 3), dtype=f32, device=edge_vec.device)
    _check(_load().e3j_harmonics_bwd(lmax, e, _dev_ptr(edge_vec, f32, (e, 3), "edge_vec"),
                                     _dev_ptr(grad_sh, f32, (e, (lmax + 1) ** 2), "grad_sh"),
                                     _dev_ptr(out, f32, (e, 3), "grad_vec"), _stream(stream)), "e3j_harmonics_bwd")
    return out


def e3j_conv_vec_fwd_workspace_bytes(plan: Plan, n_nodes: int, n_edges: int) -> int:
    return int(_load().e3j_conv_vec_fwd_workspace_bytes(plan.handle, n_nodes, n_edges))


def e3j_conv_vec_bwd_workspace_bytes(plan: Plan, n_nodes: int, n_edges: int) -> int:
    return int(_load().e3j_conv_vec_bwd_workspace_bytes(plan.handle, n_nodes, n_edges))


def e3j_conv_vec_fwd(plan: Plan, x, edge_vec, w, senders, receivers, rowptr=None, out=None, workspace=None,
                     stream=None):
    """Forward convolution with the harmonics formed from the edge vectors [E, 3]."""
    torch = _torch()
    n, e = x.shape[0], senders.numel()
    f32, i32 = torch.float32, torch.int32
    if out is None:
        out = torch.empty((n, plan.d_out, plan.n_channels), dtype=f32, device=x.device)
    workspace = _workspace(e3j_conv_vec_fwd_workspace_bytes(plan, n, e), x, workspace)
    _check(_load().e3j_conv_vec_fwd(
        plan.handle, n, e, _dev_ptr(x, f32, (n, plan.d_in, plan.n_channels), "x"),
        _dev_ptr(edge_vec, f32, (e, 3), "edge_vec"), _dev_ptr(w, f32, (e, plan.n_paths, plan.n_channels), "w"),
        _dev_ptr(senders, i32, (e,), "senders"), _dev_ptr(receivers, i32, (e,), "receivers"),
        _dev_ptr(rowptr, i32, (n + 1,), "rowptr"), _dev_ptr(out, f32, (n, plan.d_out, plan.n_channels), "out"),
        ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)), "e3j_conv_vec_fwd")
    return out


def e3j_conv_vec_bwd(plan: Plan, x, edge_vec, w, senders, receivers, grad_out, rowptr=None, sender_perm=None,
                     colptr=None, grad_x=True, grad_vec=True, grad_w=True, workspace=None, stream=None):
    """Returns (grad_x, grad_vec, grad_w); each grad_* argument is True (allocate), False/None or a tensor."""
    torch = _torch()
    n, e = x.shape[0], senders.numel()
    f32, i32 = torch.float32, torch.int32

    def alloc(flag, shape):
        if flag is True:
            return torch.empty(shape, dtype=f32, device=x.device)
        return flag if isinstance(flag, torch.Tensor) else None

    grad_x = alloc(grad_x, (n, plan.d_in, plan.n_channels))
    grad_vec = alloc(grad_vec, (e, 3))
    grad_w = alloc(grad_w, (e, plan.n_paths, plan.n_channels))
    workspace = _workspace(e3j_conv_vec_bwd_workspace_bytes(plan, n, e), x, workspace)
    _check(_load().e3j_conv_vec_bwd(
        plan.handle, n, e, _dev_ptr(x, f32, (n, plan.d_in, plan.n_channels), "x"),
        _dev_ptr(edge_vec, f32, (e, 3), "edge_vec"), _dev_ptr(w, f32, (e, plan.n_paths, plan.n_channels), "w"),
        _dev_ptr(senders, i32, (e,), "senders"), _dev_ptr(receivers, i32, (e,), "receivers"),
        _dev_ptr(rowptr, i32, (n + 1,), "rowptr"), _dev_ptr(sender_perm, i32, (e,), "sender_perm"),
        _dev_ptr(colptr, i32, (n + 1,), "colptr"),
        _dev_ptr(grad_out, f32, (n, plan.d_out, plan.n_channels), "grad_out"),
        _dev_ptr(grad_x, f32, (n, plan.d_in, plan.n_channels), "grad_x"), _dev_ptr(grad_vec, f32, (e, 3), "grad_vec"),
        _dev_ptr(grad_w, f32, (e, plan.n_paths, plan.n_channels), "grad_w"),
        ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)), "e3j_conv_vec_bwd")
    return grad_x, grad_vec, grad_w


def e3j_conv_fwd_f64(plan: Plan, x, sh, w, senders, receivers, rowptr=None, out=None, stream=None):
    """Float64 forward convolution (table-driven kernels)."""
    torch = _torch()
    n, e, f64, i32 = x.shape[0], senders.numel(), torch.float64, torch.int32
    if out is None:
        out = torch.empty((n, plan.d_out, plan.n_channels), dtype=f64, device=x.device)
    ws = _workspace(int(_load().e3j_conv_f64_workspace_bytes(plan.handle, n, e)), x, None)
    _check(_load().e3j_conv_fwd_f64(
        plan.handle, n, e, _dev_ptr(x, f64, (n, plan.d_in, plan.n_channels), "x"), _dev_ptr(sh, f64, (e, plan.d_sh), "sh"),
        _dev_ptr(w, f64, (e, plan.n_paths, plan.n_channels), "w"), _dev_ptr(senders, i32, (e,), "senders"),
        _dev_ptr(receivers, i32, (e,), "receivers"), _dev_ptr(rowptr, i32, (n + 1,), "rowptr"),
        _dev_ptr(out, f64, (n, plan.d_out, plan.n_channels), "out"), ctypes.c_void_p(ws.data_ptr()), ws.numel(),
        _stream(stream)), "e3j_conv_fwd_f64")
    return out


def e3j_conv_bwd_f64(plan: Plan, x, sh, w, senders, receivers, grad_out, sender_perm=None, colptr=None, stream=None):
    """Float64 backward convolution: (grad_x, grad_sh, grad_w)."""
    torch = _torch()
    n, e, f64, i32 = x.shape[0], senders.numel(), torch.float64, torch.int32
    gx = torch.empty((n, plan.d_in, plan.n_channels), dtype=f64, device=x.device)
    gsh = torch.empty((e, plan.d_sh), dtype=f64, device=x.device)
    gw = torch.empty((e, plan.n_paths, plan.n_channels), dtype=f64, device=x.device)
    ws = _workspace(int(_load().e3j_conv_f64_workspace_bytes(plan.handle, n, e)), x, None)
    _check(_load().e3j_conv_bwd_f64(
        plan.handle, n, e, _dev_ptr(x, f64, (n, plan.d_in, plan.n_channels), "x"), _dev_ptr(sh, f64, (e, plan.d_sh), "sh"),
        _dev_ptr(w, f64, (e, plan.n_paths, plan.n_channels), "w"), _dev_ptr(senders, i32, (e,), "senders"),
        _dev_ptr(receivers, i32, (e,), "receivers"), _dev_ptr(sender_perm, i32, (e,), "sender_perm"),
        _dev_ptr(colptr, i32, (n + 1,), "colptr"), _dev_ptr(grad_out, f64, (n, plan.d_out, plan.n_channels), "grad_out"),
        _dev_ptr(gx, f64, None, "grad_x"), _dev_ptr(gsh, f64, None, "grad_sh"), _dev_ptr(gw, f64, None, "grad_w"),
        ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream(stream)), "e3j_conv_bwd_f64")
    return gx, gsh, gw


def e3j_shard_prepare(n_nodes: int, node_lo: int, node_hi: int, senders, receivers, stream=None):
    """Local problem of the rank that owns receivers [node_lo, node_hi): (local_senders, local_receivers, halo_ids)
    for its slice of the edge list (global ids in).  halo_ids (ascending global ids) is cut to its length, which
    costs one device-to-host read of the count."""
    torch = _torch()
    e, i32 = senders.numel(), torch.int32
    dev = senders.device
    ls = torch.empty(max(e, 1), dtype=i32, device=dev)
    lr = torch.empty(max(e, 1), dtype=i32, device=dev)
    halo = torch.empty(max(n_nodes, 1), dtype=i32, device=dev)
    count = torch.zeros(1, dtype=i32, device=dev)
    ws = torch.empty(max(int(_load().e3j_shard_prepare_workspace_bytes(n_nodes)), 256), dtype=torch.uint8, device=dev)
    _check(_load().e3j_shard_prepare(n_nodes, e, node_lo, node_hi, _dev_ptr(senders, i32, (e,), "senders"),
                                     _dev_ptr(receivers, i32, (e,), "receivers"), _dev_ptr(ls, i32, None, "local_senders"),
                                     _dev_ptr(lr, i32, None, "local_receivers"), _dev_ptr(halo, i32, None, "halo_ids"),
                                     _dev_ptr(count, i32, None, "n_halo"), ctypes.c_void_p(ws.data_ptr()), ws.numel(),
                                     _stream(stream)), "e3j_shard_prepare")
    return ls[:e], lr[:e], halo[:int(count.item())]


def e3j_rows_gather(dst, src, ids, stream=None):
    """dst[i] = src[ids[i]] for float32 tensors whose trailing dimensions form the row."""
    torch = _torch()
    n = ids.numel()
    row = src[0].numel() if src.shape[0] else 0
    if n:
        _check(_load().e3j_rows_gather(_dev_ptr(dst, torch.float32, None, "dst"), _dev_ptr(src, torch.float32, None, "src"),
                                       _dev_ptr(ids, torch.int32, (n,), "ids"), n, row, _stream(stream)), "e3j_rows_gather")
    return dst


def e3j_rows_add(dst, src, ids, stream=None):
    """dst[ids[i]] += src[i]; ids must not repeat within the call."""
    torch = _torch()
    n = ids.numel()
    row = dst[0].numel() if dst.shape[0] else 0
    if n:
        _check(_load().e3j_rows_add(_dev_ptr(dst, torch.float32, None, "dst"), _dev_ptr(src, torch.float32, None, "src"),
                                    _dev_ptr(ids, torch.int32, (n,), "ids"), n, row, _stream(stream)), "e3j_rows_add")
    return dst


def e3j_selftest_bounded_wait(plan: Plan, spin_limit: int = 1000):
    """(returned, abort_flag) of a wait that is made to run out after spin_limit polls; sets the plan's status word."""
    a, b = ctypes.c_int32(-1), ctypes.c_int32(-1)
    _check(_load().e3j_selftest_bounded_wait(plan.handle, spin_limit, ctypes.byref(a), ctypes.byref(b)),
           "e3j_selftest_bounded_wait")
    return int(a.value), int(b.value)


def e3j_status_string(status: int) -> str:
    return _load().e3j_status_string(status).decode()


def e3j_launch_count() -> int:
    return int(_load().e3j_launch_count())
