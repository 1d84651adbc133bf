"""Thin ctypes binding of libgar.so: argument marshalling only.

Every function has the name and the argument order of its C entry point in
include/gar.h; tensors are passed as device (or host) pointers, the current
torch CUDA stream is used when no stream is given.  Nothing is computed here
and there is no fallback: if the library is missing, loading fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

GAR_MAX_N = 64
RULES = {"average": 0, "median": 1, "krum": 2, "multi_krum": 3, "bulyan": 4, "multi_bulyan": 5}
EVEN_MEDIAN = {"lower": 0, "mean": 1}
DISTANCE_MODES = {"auto": 0, "difference": 1}
GRAD_DTYPES = {torch.float32: 0, torch.bfloat16: 1, torch.float16: 2}
# gar_workspace control block, word 4: how the last distance call ran
DISTANCE_PATHS = {0: "difference", 1: "gram", 2: "gram_rejected"}
GAR_OK = 0
GAR_ERR_CUDA = 5
STATUS_NAMES = {0: "GAR_OK", 1: "GAR_ERR_INVALID_ARG", 2: "GAR_ERR_PRECONDITION", 3: "GAR_ERR_UNSUPPORTED",
                4: "GAR_ERR_WORKSPACE", 5: "GAR_ERR_CUDA", 6: "GAR_ERR_TIMEOUT"}

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libgar.so")
_lib = None


class GarSelection(C.Structure):
    """Mirror of gar_selection_t."""
    _fields_ = [
        ("n", C.c_int32), ("f", C.c_int32), ("rule", C.c_int32), ("theta", C.c_int32), ("beta", C.c_int32),
        ("preagg", C.c_int32), ("median_of_agr", C.c_int32), ("status", C.c_int32),
        ("even_median", C.c_int32), ("reserved", C.c_int32),
        ("winners", C.c_int32 * GAR_MAX_N),
        ("m", C.c_int32 * GAR_MAX_N),
        ("sets", C.c_uint64 * GAR_MAX_N),
        ("gap_winner", C.c_double * GAR_MAX_N),
        ("gap_set", C.c_double * GAR_MAX_N),
        ("nu", C.c_int32), ("total_adds", C.c_int32), ("nbase", C.c_int32), ("nloose", C.c_int32),
        ("chain_mask", C.c_uint64), ("corr_mask", C.c_uint64),
        ("base_rows", C.c_uint8 * GAR_MAX_N),
        ("loose_rows", C.c_uint8 * GAR_MAX_N),
        ("slot_src", C.c_uint8 * GAR_MAX_N),
        ("slot_save", C.c_uint8 * GAR_MAX_N),
        ("slot_nadd", C.c_uint8 * GAR_MAX_N),
        ("add_pos", C.c_uint8 * (GAR_MAX_N * GAR_MAX_N)),
        ("scores", (C.c_double * GAR_MAX_N) * GAR_MAX_N),
    ]


class GarParams(C.Structure):
    """Mirror of gar_params_t."""
    _fields_ = [
        ("rule", C.c_int32), ("n", C.c_int32), ("f", C.c_int32),
        ("d", C.c_int64), ("ld", C.c_int64),
        ("grads", C.c_void_p), ("out", C.c_void_p), ("stream", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("m", C.c_int32), ("theta", C.c_int32), ("median_of_agr", C.c_int32), ("even_median", C.c_int32),
        ("dist_out", C.c_void_p), ("selection_out", C.c_void_p),
        ("distance_mode", C.c_int32), ("grads_dtype", C.c_int32),
        ("sgd_params", C.c_void_p), ("sgd_momentum_buf", C.c_void_p), ("sgd_lr", C.c_float), ("sgd_momentum", C.c_float),
    ]


class GarTensor(C.Structure):
    """Mirror of gar_tensor_t."""
    _fields_ = [("grads", C.c_void_p), ("out", C.c_void_p), ("d", C.c_int64), ("ld", C.c_int64),
                ("sgd_params", C.c_void_p), ("sgd_momentum_buf", C.c_void_p)]


class GarMultiParams(C.Structure):
    """Mirror of gar_multi_params_t."""
    _fields_ = [
        ("rule", C.c_int32), ("n", C.c_int32), ("f", C.c_int32), ("count", C.c_int32),
        ("joint", C.c_int32), ("even_median", C.c_int32),
        ("tensors", C.POINTER(GarTensor)), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("dist_out", C.c_void_p), ("selection_out", C.c_void_p), ("stream", C.c_void_p),
        ("sgd_lr", C.c_float), ("sgd_momentum", C.c_float), ("grads_dtype", C.c_int32),
    ]


class GarError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().gar_status_string(status).decode()
        if status == GAR_ERR_CUDA:
            msg += f": {gar_last_cuda_error()[1]}"
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({msg})")


def lib():
    """The loaded library.  Raises if libgar.so has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with "
                               "`python -m paper_1905_04374_b200.build` (needs nvcc); there is no fallback")
        L = C.CDLL(_LIB_PATH)
        L.gar_version.restype = C.c_int
        L.gar_status_string.restype = C.c_char_p
        L.gar_status_string.argtypes = [C.c_int]
        L.gar_last_cuda_error.restype = C.c_int
        L.gar_last_cuda_error_name.restype = C.c_char_p
        L.gar_theta.argtypes = [C.c_int, C.c_int, C.c_int]
        L.gar_beta.argtypes = [C.c_int, C.c_int, C.c_int]
        L.gar_workspace_bytes.restype = C.c_size_t
        L.gar_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int64]
        L.gar_aggregate.argtypes = [C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int64, C.c_void_p, C.c_void_p]
        L.gar_aggregate_ex.argtypes = [C.POINTER(GarParams)]
        L.gar_aggregate_host.argtypes = [C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int64, C.c_void_p]
        L.gar_pairwise_distances.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                             C.c_size_t, C.c_void_p]
        L.gar_pairwise_distances_mode.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                                  C.c_size_t, C.c_int, C.c_void_p]
        L.gar_reduce_partials.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.gar_multi_workspace_bytes.restype = C.c_size_t
        L.gar_multi_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int]
        L.gar_aggregate_multi.argtypes = [C.POINTER(GarMultiParams)]
        L.gar_selftest_bounded_wait.argtypes = [C.c_uint, C.c_void_p, C.c_void_p]
        L.gar_pairwise_distances_static.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p]
        L.gar_select.argtypes = [C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                 C.c_void_p, C.c_void_p]
        L.gar_schedule_from_tables.argtypes = [C.c_void_p, C.c_void_p]
        L.gar_coordinate_phase.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_void_p, C.c_int, C.c_int,
                                           C.c_void_p, C.c_void_p]
        L.gar_shutdown.restype = None
        _lib = L
    return _lib


def _rule(rule) -> int:
    return RULES[rule] if isinstance(rule, str) else int(rule)


def _even(even_median) -> int:
    return EVEN_MEDIAN[even_median] if isinstance(even_median, str) else int(even_median)


def _mode(distance_mode) -> int:
    return DISTANCE_MODES[distance_mode] if isinstance(distance_mode, str) else int(distance_mode)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(status: int, where: str):
    if status != GAR_OK:
        raise GarError(status, where)


def _dev_f32(t: torch.Tensor, name: str):
    if not (t.is_cuda and t.dtype == torch.float32):
        raise TypeError(f"{name} must be a CUDA float32 tensor")
    return t


def gar_version() -> int:
    return lib().gar_version()


def gar_status_string(status: int) -> str:
    return lib().gar_status_string(status).decode()


def gar_last_cuda_error():
    """(cudaError_t value, the runtime's name for it) behind this thread's latest GAR_ERR_CUDA."""
    return lib().gar_last_cuda_error(), lib().gar_last_cuda_error_name().decode()


def gar_theta(rule, n: int, f: int) -> int:
    return lib().gar_theta(_rule(rule), n, f)


def gar_beta(rule, n: int, f: int) -> int:
    return lib().gar_beta(_rule(rule), n, f)


def gar_workspace_bytes(rule, n: int, f: int, d: int) -> int:
    return lib().gar_workspace_bytes(_rule(rule), n, f, d)


def _rows(grads: torch.Tensor):
    """(n, d, ld) of a 2-D tensor whose rows are contiguous."""
    if grads.dim() != 2 or grads.stride(1) != 1:
        raise ValueError("grads must be 2-D with unit column stride")
    n, d = grads.shape
    ld = grads.stride(0) if n > 1 else d
    return n, d, ld


def gar_aggregate(rule, grads: torch.Tensor, f: int, out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """gar_aggregate: grads CUDA fp32 [n, d] contiguous, returns out [d]."""
    _dev_f32(grads, "grads")
    n, d, ld = _rows(grads)
    if ld != d:
        raise ValueError("gar_aggregate needs contiguous rows; use gar_aggregate_ex for a row stride")
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=grads.device)
    _dev_f32(out, "out")
    with torch.cuda.device(grads.device):
        st = lib().gar_aggregate(_rule(rule), grads.data_ptr(), n, f, d, out.data_ptr(), _stream(stream))
    _check(st, "gar_aggregate")
    return out


def gar_aggregate_ex(rule, grads: torch.Tensor, f: int, out: torch.Tensor | None = None, stream=None,
                     workspace: torch.Tensor | None = None, m: int = 0, theta: int = 0, median_of_agr: int = 0,
                     dist_out: torch.Tensor | None = None, selection_out: torch.Tensor | None = None,
                     even_median=0, distance_mode=0, sgd_params: torch.Tensor | None = None,
                     sgd_momentum_buf: torch.Tensor | None = None, sgd_lr: float = 0.0, sgd_momentum: float = 0.0,
                     store_out: bool = True):
    """gar_aggregate_ex: row stride taken from the tensor; optional workspace
    (uint8 CUDA tensor), options and outputs (dist_out float64 [n, n];
    selection_out uint8 CUDA tensor of sizeof(gar_selection_t)); optional fused SGD step on
    sgd_params / sgd_momentum_buf (CUDA float32 [d], updated in place); store_out=False with a
    fused step passes out = NULL (returns None).  grads may be float32, bfloat16 or float16."""
    if not (grads.is_cuda and grads.dtype in GRAD_DTYPES):
        raise TypeError("grads must be a CUDA float32, bfloat16 or float16 tensor")
    n, d, ld = _rows(grads)
    if out is None and (store_out or sgd_params is None):
        out = torch.empty(d, dtype=torch.float32, device=grads.device)
    p = GarParams()
    p.rule, p.n, p.f, p.d, p.ld = _rule(rule), n, f, d, ld
    p.grads, p.stream = grads.data_ptr(), _stream(stream)
    p.out = out.data_ptr() if out is not None else None
    if sgd_params is not None:
        p.sgd_params = _dev_f32(sgd_params, "sgd_params").data_ptr()
        p.sgd_lr, p.sgd_momentum = sgd_lr, sgd_momentum
    if sgd_momentum_buf is not None:
        p.sgd_momentum_buf = _dev_f32(sgd_momentum_buf, "sgd_momentum_buf").data_ptr()
    if workspace is not None:
        p.workspace, p.workspace_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    p.m, p.theta, p.median_of_agr = m, theta, median_of_agr
    p.even_median, p.distance_mode = _even(even_median), _mode(distance_mode)
    p.grads_dtype = GRAD_DTYPES[grads.dtype]
    if dist_out is not None:
        p.dist_out = dist_out.data_ptr()
    if selection_out is not None:
        p.selection_out = selection_out.data_ptr()
    with torch.cuda.device(grads.device):
        st = lib().gar_aggregate_ex(C.byref(p))
    _check(st, "gar_aggregate_ex")
    return out


def gar_multi_workspace_bytes(rule, n: int, f: int, count: int) -> int:
    return lib().gar_multi_workspace_bytes(_rule(rule), n, f, count)


def gar_aggregate_multi(rule, grads, f: int, outs=None, joint: bool = False, even_median=0, workspace=None,
                        dist_out: torch.Tensor | None = None, selection_out: torch.Tensor | None = None, stream=None,
                        sgd_params=None, sgd_momentum_bufs=None, sgd_lr: float = 0.0, sgd_momentum: float = 0.0,
                        store_out: bool = True):
    """gar_aggregate_multi: `grads` is a list of CUDA float32 (or all bfloat16 / all float16) tensors
    [n, d_t] (one per layer, the same n, unit column stride); returns the list of aggregates [d_t].  joint=False: every tensor
    is a problem of its own; joint=True: the tensors are the pieces of one gradient (one selection).
    Optional: workspace (uint8 CUDA tensor of gar_multi_workspace_bytes), dist_out float64
    [count, n, n] ([n, n] when joint), selection_out uint8 CUDA tensor of count (1 when joint)
    times sizeof(gar_selection_t); a fused SGD step on the lists sgd_params / sgd_momentum_bufs
    (CUDA float32 [d_t] each, updated in place; store_out=False then passes out = NULL and
    returns None)."""
    grads = list(grads)
    if not grads:
        raise ValueError("grads is empty")
    dev = grads[0].device
    n = grads[0].shape[0]
    count = len(grads)
    if outs is None and (store_out or sgd_params is None):
        outs = [torch.empty(g.shape[1], dtype=torch.float32, device=dev) for g in grads]
    tensors = (GarTensor * count)()
    dtype = grads[0].dtype
    if dtype not in GRAD_DTYPES:
        raise TypeError("grads must be float32, bfloat16 or float16 tensors")
    for t, g in enumerate(grads):
        if not (g.is_cuda and g.dtype == dtype):
            raise TypeError("grads[%d] must be a CUDA tensor of the same element type as grads[0]" % t)
        gn, d, ld = _rows(g)
        if gn != n or g.device != dev:
            raise ValueError("every tensor must have the same number of rows and sit on the same device")
        tensors[t].grads, tensors[t].d, tensors[t].ld = g.data_ptr(), d, ld
        vecs = {"out": outs[t] if outs is not None else None,
                "sgd_params": sgd_params[t] if sgd_params is not None else None,
                "sgd_momentum_buf": sgd_momentum_bufs[t] if sgd_momentum_bufs is not None else None}
        for name, o in vecs.items():
            if o is None:
                continue
            if not (o.is_cuda and o.dtype == torch.float32 and o.is_contiguous() and o.numel() == d):
                raise TypeError("%s[%d] must be a contiguous CUDA float32 tensor of d elements" % (name, t))
            setattr(tensors[t], name, o.data_ptr())
    if workspace is None:
        workspace = torch.empty(gar_multi_workspace_bytes(rule, n, f, count), dtype=torch.uint8, device=dev)
    p = GarMultiParams()
    p.rule, p.n, p.f, p.count = _rule(rule), n, f, count
    p.joint, p.even_median = 1 if joint else 0, _even(even_median)
    p.tensors = tensors
    p.workspace, p.workspace_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    if dist_out is not None:
        p.dist_out = dist_out.data_ptr()
    if selection_out is not None:
        p.selection_out = selection_out.data_ptr()
    p.stream = _stream(stream)
    p.sgd_lr, p.sgd_momentum = sgd_lr, sgd_momentum
    p.grads_dtype = GRAD_DTYPES[dtype]
    with torch.cuda.device(dev):
        st = lib().gar_aggregate_multi(C.byref(p))
    _check(st, "gar_aggregate_multi")
    return outs


def gar_aggregate_host(rule, grads: torch.Tensor, f: int, out: torch.Tensor | None = None) -> torch.Tensor:
    """gar_aggregate_host: grads and out are HOST fp32 tensors (pinned for speed)."""
    if grads.is_cuda or grads.dtype != torch.float32 or not grads.is_contiguous():
        raise TypeError("grads must be a contiguous host float32 tensor")
    n, d = grads.shape
    if out is None:
        out = torch.empty(d, dtype=torch.float32, pin_memory=grads.is_pinned())
    st = lib().gar_aggregate_host(_rule(rule), grads.data_ptr(), n, f, d, out.data_ptr())
    _check(st, "gar_aggregate_host")
    return out


def gar_pairwise_distances(grads: torch.Tensor, dist: torch.Tensor | None = None, workspace=None,
                           stream=None, distance_mode=0) -> torch.Tensor:
    """gar_pairwise_distances (gar_pairwise_distances_mode when a mode is given): returns dist
    float64 [n, n] on the device."""
    _dev_f32(grads, "grads")
    n, d, ld = _rows(grads)
    if dist is None:
        dist = torch.empty(n, n, dtype=torch.float64, device=grads.device)
    wp, wb = (workspace.data_ptr(), workspace.numel() * workspace.element_size()) if workspace is not None else (None, 0)
    with torch.cuda.device(grads.device):
        if _mode(distance_mode) == 0:
            st = lib().gar_pairwise_distances(grads.data_ptr(), n, d, ld, dist.data_ptr(), wp, wb, _stream(stream))
        else:
            st = lib().gar_pairwise_distances_mode(grads.data_ptr(), n, d, ld, dist.data_ptr(), wp, wb,
                                                   _mode(distance_mode), _stream(stream))
    _check(st, "gar_pairwise_distances")
    return dist


def gar_reduce_partials(parts: torch.Tensor, dist: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """gar_reduce_partials: parts CUDA float64 [count, n, n] -> dist [n, n] = parts[0] + parts[1] + ... in order."""
    if not (parts.is_cuda and parts.dtype == torch.float64 and parts.is_contiguous() and parts.dim() == 3):
        raise TypeError("parts must be a contiguous CUDA float64 tensor [count, n, n]")
    count, n, _ = parts.shape
    if dist is None:
        dist = torch.empty(n, n, dtype=torch.float64, device=parts.device)
    with torch.cuda.device(parts.device):
        st = lib().gar_reduce_partials(parts.data_ptr(), count, n, dist.data_ptr(), _stream(stream))
    _check(st, "gar_reduce_partials")
    return dist


def distance_path(workspace: torch.Tensor) -> str:
    """How the last distance call that used this caller-owned workspace ran (control block, word 4)."""
    word = workspace[16:20].cpu().numpy().view("uint32")[0]
    return DISTANCE_PATHS.get(int(word), str(int(word)))


def gar_selftest_bounded_wait(limit: int, device="cuda", stream=None):
    """gar_selftest_bounded_wait: (status, nanoseconds) of a bounded wait on a barrier nobody arrives on."""
    res = torch.zeros(2, dtype=torch.int64, device=device)
    with torch.cuda.device(res.device):
        st = lib().gar_selftest_bounded_wait(limit, res.data_ptr(), _stream(stream))
    _check(st, "gar_selftest_bounded_wait")
    host = res.cpu()
    return int(host[0]), int(host[1])


def gar_pairwise_distances_static(grads: torch.Tensor, dist: torch.Tensor, stream=None) -> torch.Tensor:
    """gar_pairwise_distances_static: the distance step with no allocation inside the library.
    The caller supplies `dist` (CUDA float64 [n, n]); this wrapper allocates nothing either."""
    _dev_f32(grads, "grads")
    n, d, ld = _rows(grads)
    if not (dist.is_cuda and dist.dtype == torch.float64 and dist.is_contiguous() and dist.numel() == n * n):
        raise TypeError("dist must be a contiguous CUDA float64 tensor with n*n elements")
    with torch.cuda.device(grads.device):
        st = lib().gar_pairwise_distances_static(grads.data_ptr(), n, d, ld, dist.data_ptr(), _stream(stream))
    _check(st, "gar_pairwise_distances_static")
    return dist


def new_selection(device) -> torch.Tensor:
    """Device buffer for one gar_selection_t."""
    return torch.zeros(C.sizeof(GarSelection), dtype=torch.uint8, device=device)


def read_selection(sel: torch.Tensor) -> GarSelection:
    """Copy a device gar_selection_t to the host."""
    raw = sel.cpu().numpy().tobytes()
    return GarSelection.from_buffer_copy(raw)


def write_selection(host: GarSelection, device) -> torch.Tensor:
    """Upload a host gar_selection_t."""
    import numpy as np
    arr = np.frombuffer(bytes(host), dtype=np.uint8).copy()
    return torch.from_numpy(arr).to(device)


def gar_select(rule, dist: torch.Tensor | None, n: int, f: int, m: int = 0, theta: int = 0, median_of_agr: int = 0,
               sel: torch.Tensor | None = None, stream=None, device=None, even_median=0) -> torch.Tensor:
    """gar_select: dist CUDA float64 [n, n]; returns the device gar_selection_t buffer."""
    device = dist.device if dist is not None else (device or "cuda")
    if sel is None:
        sel = new_selection(device)
    dp = None
    if dist is not None:
        if not (dist.is_cuda and dist.dtype == torch.float64 and dist.is_contiguous()):
            raise TypeError("dist must be a contiguous CUDA float64 tensor")
        dp = dist.data_ptr()
    with torch.cuda.device(sel.device):
        st = lib().gar_select(_rule(rule), dp, n, f, m, theta, median_of_agr, _even(even_median), sel.data_ptr(),
                              _stream(stream))
    _check(st, "gar_select")
    return sel


def gar_schedule_from_tables(sel: torch.Tensor, stream=None) -> torch.Tensor:
    with torch.cuda.device(sel.device):
        st = lib().gar_schedule_from_tables(sel.data_ptr(), _stream(stream))
    _check(st, "gar_schedule_from_tables")
    return sel


def gar_coordinate_phase(grads: torch.Tensor, sel: torch.Tensor, theta: int, preagg: int,
                         out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    _dev_f32(grads, "grads")
    n, d, ld = _rows(grads)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=grads.device)
    with torch.cuda.device(grads.device):
        st = lib().gar_coordinate_phase(grads.data_ptr(), n, d, ld, sel.data_ptr(), theta, preagg, out.data_ptr(),
                                        _stream(stream))
    _check(st, "gar_coordinate_phase")
    return out


def gar_shutdown() -> None:
    lib().gar_shutdown()
