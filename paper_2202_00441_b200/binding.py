"""ctypes binding of include/fewbit.h -- argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libfewbit.so")

ACTS = {"gelu": 0, "silu": 1, "sigmoid": 2, "tanh": 3, "elu": 4, "softplus": 5, "leaky_relu": 6,
        "relu": 7, "selu": 8}
_DTYPES = {torch.float32: 0, torch.bfloat16: 1, torch.float16: 2}

_lib = None


class FewbitError(RuntimeError):
    def __init__(self, status: int, where: str):
        msg = load_library().fewbit_status_string(status).decode()
        extra = ""
        if status == 4:
            extra = f" (cudaError {load_library().fewbit_last_cuda_error()})"
        super().__init__(f"{where}: {msg}{extra}")
        self.status = status


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads libfewbit.so; raises if it has not been built (no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2202_00441_b200.build` "
            "(nvcc, sm_100a); this package has no other execution path")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
    lib.fewbit_table_create.restype = vp
    lib.fewbit_table_create.argtypes = [ci, ci]
    lib.fewbit_table_create_ex.restype = ci
    lib.fewbit_table_create_ex.argtypes = [ci, ci, ctypes.c_double, ctypes.c_double, ci, ctypes.POINTER(vp)]
    lib.fewbit_table_from_arrays.restype = ci
    lib.fewbit_table_from_arrays.argtypes = [ci, ci, vp, vp, ctypes.POINTER(vp)]
    lib.fewbit_table_create_folded.restype = ci
    lib.fewbit_table_create_folded.argtypes = [ci, ci, ctypes.c_double, ci, ctypes.POINTER(vp)]
    lib.fewbit_table_from_arrays_ex.restype = ci
    lib.fewbit_table_from_arrays_ex.argtypes = [ci, ci, vp, vp, ci, ctypes.POINTER(vp)]
    lib.fewbit_table_create_opt.restype = ci
    lib.fewbit_table_create_opt.argtypes = [ci, ci, vp, ctypes.POINTER(vp)]
    lib.fewbit_table_is_folded.restype = ci
    lib.fewbit_table_is_folded.argtypes = [vp]
    lib.fewbit_table_destroy.restype = None
    lib.fewbit_table_destroy.argtypes = [vp]
    lib.fewbit_table_get.restype = ci
    lib.fewbit_table_get.argtypes = [vp, ctypes.POINTER(ci), ctypes.POINTER(ci), vp, vp, ctypes.POINTER(ctypes.c_double)]
    lib.fewbit_packed_bytes.restype = sz
    lib.fewbit_packed_bytes.argtypes = [sz, ci]
    lib.fewbit_fwd.restype = ci
    lib.fewbit_fwd.argtypes = [vp, vp, vp, vp, sz, ci, vp]
    lib.fewbit_fwd_bias.restype = ci
    lib.fewbit_fwd_bias.argtypes = [vp, vp, vp, vp, vp, sz, sz, ci, vp]
    lib.fewbit_bwd.restype = ci
    lib.fewbit_bwd.argtypes = [vp, vp, vp, vp, sz, ci, vp]
    lib.fewbit_host_workspace_bytes.restype = sz
    lib.fewbit_host_workspace_bytes.argtypes = [sz, ci, ci]
    lib.fewbit_fwd_host.restype = ci
    lib.fewbit_fwd_host.argtypes = [vp, vp, vp, vp, sz, ci, vp, sz]
    lib.fewbit_bwd_host.restype = ci
    lib.fewbit_bwd_host.argtypes = [vp, vp, vp, vp, sz, ci, vp, sz]
    lib.fewbit_static_max_elements.restype = sz
    lib.fewbit_static_max_elements.argtypes = []
    lib.fewbit_fwd_host_static.restype = ci
    lib.fewbit_fwd_host_static.argtypes = [vp, vp, vp, vp, sz, ci, vp]
    lib.fewbit_status_string.restype = ctypes.c_char_p
    lib.fewbit_status_string.argtypes = [ci]
    lib.fewbit_last_cuda_error.restype = ci
    lib.fewbit_last_cuda_error.argtypes = []
    lib.fewbit_launch_count.restype = ctypes.c_uint64
    lib.fewbit_launch_count.argtypes = []
    lib.fewbit_set_option.restype = ci
    lib.fewbit_set_option.argtypes = [ci, ci]
    lib.fewbit_get_option.restype = ci
    lib.fewbit_get_option.argtypes = [ci]
    lib.fewbit_tail_warp_count.restype = ci
    lib.fewbit_tail_warp_count.argtypes = [ctypes.POINTER(ctypes.c_uint64), ci]
    lib.fewbit_f32_activation_scan.restype = ci
    lib.fewbit_f32_activation_scan.argtypes = [ci, ctypes.c_uint64, ctypes.c_uint64, vp, vp]
    _lib = lib
    return lib


def _check(status: int, where: str) -> None:
    if status != 0:
        raise FewbitError(status, where)


def _act_id(act) -> int:
    return ACTS[act] if isinstance(act, str) else int(act)


class Table:
    """Owns a ``fewbit_table*`` (host object: K-1 boundaries, K levels)."""

    def __init__(self, handle: int):
        if not handle:
            raise FewbitError(1, "fewbit_table_create")
        self._h = ctypes.c_void_p(handle)
        act, bits, obj = ctypes.c_int(), ctypes.c_int(), ctypes.c_double()
        _check(load_library().fewbit_table_get(self._h, ctypes.byref(act), ctypes.byref(bits), None, None,
                                               ctypes.byref(obj)), "fewbit_table_get")
        self.act, self.bits, self.objective = act.value, bits.value, obj.value
        self.folded = bool(load_library().fewbit_table_is_folded(self._h))

    @property
    def handle(self):
        return self._h

    def arrays(self):
        """(s, lev) as float32 numpy arrays, read back through the C ABI."""
        import numpy as np

        K = 1 << self.bits
        s = np.zeros(max(K - 1, 1), dtype=np.float32)
        lev = np.zeros(K, dtype=np.float32)
        _check(load_library().fewbit_table_get(self._h, None, None, s.ctypes.data, lev.ctypes.data, None),
               "fewbit_table_get")
        return s[:K - 1].copy(), lev

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h and _lib is not None:
            _lib.fewbit_table_destroy(h)


def fewbit_table_create(act, bits: int) -> Table:
    return Table(load_library().fewbit_table_create(_act_id(act), int(bits)) or 0)


def fewbit_table_create_ex(act, bits: int, A: float, B: float, n_cells: int) -> Table:
    out = ctypes.c_void_p()
    _check(load_library().fewbit_table_create_ex(_act_id(act), int(bits), float(A), float(B), int(n_cells),
                                                 ctypes.byref(out)), "fewbit_table_create_ex")
    return Table(out.value or 0)


def fewbit_table_create_folded(act, bits: int, B: float = 8.0, n_cells: int = 2048) -> Table:
    """Folded table (even derivative: sigmoid, tanh): 2^bits pieces on [0, B], codes from |x|."""
    out = ctypes.c_void_p()
    _check(load_library().fewbit_table_create_folded(_act_id(act), int(bits), float(B), int(n_cells),
                                                     ctypes.byref(out)), "fewbit_table_create_folded")
    return Table(out.value or 0)


class _SolverOptions(ctypes.Structure):
    _fields_ = [("A", ctypes.c_double), ("B", ctypes.c_double), ("n_cells", ctypes.c_int), ("weight", ctypes.c_int),
                ("finetune_iters", ctypes.c_int), ("folded", ctypes.c_int)]


def fewbit_table_create_opt(act, bits: int, A: float = -8.0, B: float = 8.0, n_cells: int = 4096,
                            weight: str = "uniform", finetune_iters: int = 0, folded: bool = False) -> Table:
    """Solver with explicit options: weight "uniform" | "normal" (Eq. 3), gradient fine-tuning (Eq. 5)."""
    opt = _SolverOptions(float(A), float(B), int(n_cells), {"uniform": 0, "normal": 1}[weight], int(finetune_iters),
                         int(bool(folded)))
    out = ctypes.c_void_p()
    _check(load_library().fewbit_table_create_opt(_act_id(act), int(bits), ctypes.byref(opt), ctypes.byref(out)),
           "fewbit_table_create_opt")
    return Table(out.value or 0)


def fewbit_table_from_arrays(act, bits: int, s, lev, folded: bool = False) -> Table:
    import numpy as np

    s = np.ascontiguousarray(s, dtype=np.float32)
    lev = np.ascontiguousarray(lev, dtype=np.float32)
    K = 1 << int(bits)
    if s.size != K - 1 or lev.size != K:
        raise ValueError("need 2^bits - 1 boundaries and 2^bits levels")
    if s.size == 0:
        s = np.zeros(1, dtype=np.float32)
    out = ctypes.c_void_p()
    _check(load_library().fewbit_table_from_arrays_ex(_act_id(act), int(bits), s.ctypes.data, lev.ctypes.data,
                                                      int(bool(folded)), ctypes.byref(out)), "fewbit_table_from_arrays")
    return Table(out.value or 0)


def fewbit_packed_bytes(n: int, bits: int) -> int:
    return int(load_library().fewbit_packed_bytes(int(n), int(bits)))


def fewbit_launch_count() -> int:
    return int(load_library().fewbit_launch_count())


OPTIONS = {"fwd_table": 0, "fwd_queue": 1, "fwd_iters": 2, "fwd_warps": 3, "pdl": 4, "count_tails": 5, "fwd_tile": 6}
_OPTION_VALUES = {"auto": 0, "always": 1, "never": 2}


def fewbit_set_option(option, value) -> None:
    """Process-wide testing / tuning switch; `option` by name or number, `value` an int (for
    "fwd_table" and "fwd_tile" also "auto" | "always" | "never"; for "fwd_queue" "auto" | "never")."""
    opt = OPTIONS[option] if isinstance(option, str) else int(option)
    if isinstance(value, str):
        value = {"auto": 0, "never": 1}[value] if opt == 1 else _OPTION_VALUES[value]
    _check(load_library().fewbit_set_option(opt, int(value)), "fewbit_set_option")


def fewbit_get_option(option) -> int:
    return int(load_library().fewbit_get_option(OPTIONS[option] if isinstance(option, str) else int(option)))


def fewbit_tail_warp_count(device=None, reset: bool = False) -> int:
    """Warps that ran the forward kernel's ragged-tail path on `device` while the "count_tails"
    option was on.  Synchronises the device."""
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    out = ctypes.c_uint64()
    with torch.cuda.device(device):
        _check(load_library().fewbit_tail_warp_count(ctypes.byref(out), int(reset)), "fewbit_tail_warp_count")
    return int(out.value)


def fewbit_f32_activation_scan(act, first_pattern: int = 0, count: int = 1 << 32, device=None,
                               stream: Optional[torch.cuda.Stream] = None) -> dict:
    """Accuracy of the binary32 evaluation of `act` against its binary64 form over a range of input
    bit patterns (default: all of them).  Returns {"hist": [n0, n1, n2, n_more], "max_ulp": d,
    "worst_pattern": bits}."""
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    res = torch.zeros(5, dtype=torch.int64, device=device)
    with torch.cuda.device(device):
        _check(load_library().fewbit_f32_activation_scan(_act_id(act), int(first_pattern), int(count), res.data_ptr(),
                                                          _stream_ptr(stream, device)), "fewbit_f32_activation_scan")
        (stream or torch.cuda.current_stream(device)).synchronize()
    v = [int(a) & 0xFFFFFFFFFFFFFFFF for a in res.cpu().tolist()]
    return {"hist": v[:4], "max_ulp": v[4] >> 32, "worst_pattern": v[4] & 0xFFFFFFFF}


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)    # the current stream's handle without building a Stream object


def _stream_ptr(stream: Optional[torch.cuda.Stream], device) -> int:
    if stream is not None:
        return stream.cuda_stream
    if _raw_stream is not None and device.index is not None:
        return _raw_stream(device.index)
    return torch.cuda.current_stream(device).cuda_stream


class _NoSwitch:
    def __enter__(self):
        return None

    def __exit__(self, *exc):
        return False


_NO_SWITCH = _NoSwitch()


def _current(device):
    """Context that makes `device` current for the call; free when it already is (a launch on a
    small tensor costs less than torch.cuda.device's own bookkeeping)."""
    if device.index is None or device.index == torch.cuda.current_device():
        return _NO_SWITCH
    return torch.cuda.device(device)


def _packed_bytes(n: int, bits: int) -> int:
    return 4 * ((n * bits + 31) // 32)          # fewbit_packed_bytes without the foreign call


def _dev_tensor(t: torch.Tensor, name: str) -> torch.Tensor:
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor")
    return t


def fewbit_fwd(table: Table, x: torch.Tensor, y: Optional[torch.Tensor] = None,
               packed: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Forward half on device tensors; returns (y, packed).  ``packed`` is an
    int32 tensor of ``fewbit_packed_bytes(n, bits) / 4`` words."""
    lib = load_library()
    _dev_tensor(x, "x")
    n = x.numel()
    if y is None:
        y = torch.empty_like(x)
    if packed is None:
        packed = torch.empty(_packed_bytes(n, table.bits) // 4, dtype=torch.int32, device=x.device)
    _dev_tensor(y, "y"), _dev_tensor(packed, "packed")
    if y.dtype != x.dtype or y.numel() != n or packed.numel() * packed.element_size() < _packed_bytes(n, table.bits):
        raise ValueError("y / packed do not match x")
    with _current(x.device):
        _check(lib.fewbit_fwd(table.handle, x.data_ptr(), y.data_ptr(), packed.data_ptr(), n, _DTYPES[x.dtype],
                              _stream_ptr(stream, x.device)), "fewbit_fwd")
    return y, packed


def fewbit_fwd_bias(table: Table, x: torch.Tensor, bias: torch.Tensor, y: Optional[torch.Tensor] = None,
                    packed: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Forward half of ``f(x + bias)``: ``bias`` has one value per element of the last dimension of
    ``x`` (a multiple of 8); returns (y, packed) exactly as ``fewbit_fwd`` would for the tensor
    ``x + bias`` rounded to the storage type."""
    lib = load_library()
    _dev_tensor(x, "x"), _dev_tensor(bias, "bias")
    n, cols = x.numel(), bias.numel()
    if bias.dtype != x.dtype or x.dim() == 0 or x.shape[-1] != cols:
        raise ValueError("bias must have the dtype of x and the length of its last dimension")
    rows = n // cols if cols else 0
    if y is None:
        y = torch.empty_like(x)
    if packed is None:
        packed = torch.empty(_packed_bytes(n, table.bits) // 4, dtype=torch.int32, device=x.device)
    _dev_tensor(y, "y"), _dev_tensor(packed, "packed")
    if y.dtype != x.dtype or y.numel() != n or packed.numel() * packed.element_size() < _packed_bytes(n, table.bits):
        raise ValueError("y / packed do not match x")
    with _current(x.device):
        _check(lib.fewbit_fwd_bias(table.handle, x.data_ptr(), bias.data_ptr(), y.data_ptr(), packed.data_ptr(), rows, cols,
                                   _DTYPES[x.dtype], _stream_ptr(stream, x.device)), "fewbit_fwd_bias")
    return y, packed


def fewbit_bwd(table: Table, packed: torch.Tensor, grad_out: torch.Tensor,
               grad_in: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Backward half on device tensors; returns grad_in."""
    lib = load_library()
    _dev_tensor(grad_out, "grad_out"), _dev_tensor(packed, "packed")
    n = grad_out.numel()
    if grad_in is None:
        grad_in = torch.empty_like(grad_out)
    _dev_tensor(grad_in, "grad_in")
    if grad_in.dtype != grad_out.dtype or grad_in.numel() != n or \
            packed.numel() * packed.element_size() < _packed_bytes(n, table.bits):
        raise ValueError("grad_in / packed do not match grad_out")
    with _current(grad_out.device):
        _check(lib.fewbit_bwd(table.handle, packed.data_ptr(), grad_out.data_ptr(), grad_in.data_ptr(), n,
                              _DTYPES[grad_out.dtype], _stream_ptr(stream, grad_out.device)), "fewbit_bwd")
    return grad_in


def fewbit_host_workspace_bytes(chunk_elems: int, dtype: torch.dtype, bits: int) -> int:
    return int(load_library().fewbit_host_workspace_bytes(int(chunk_elems), _DTYPES[dtype], int(bits)))


def _host_tensor(t: torch.Tensor, name: str) -> torch.Tensor:
    if t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous host tensor")
    return t


def fewbit_fwd_host(table: Table, x: torch.Tensor, y: torch.Tensor, packed: torch.Tensor, workspace: torch.Tensor):
    """Forward half on host tensors (pinned for full speed), streamed through
    the device ``workspace`` (a uint8 CUDA tensor).  Blocks until done."""
    lib = load_library()
    _host_tensor(x, "x"), _host_tensor(y, "y"), _host_tensor(packed, "packed"), _dev_tensor(workspace, "workspace")
    n = x.numel()
    if y.dtype != x.dtype or y.numel() != n or packed.numel() * packed.element_size() < fewbit_packed_bytes(n, table.bits):
        raise ValueError("y / packed do not match x")
    with torch.cuda.device(workspace.device):
        _check(lib.fewbit_fwd_host(table.handle, x.data_ptr(), y.data_ptr(), packed.data_ptr(), n, _DTYPES[x.dtype],
                                   workspace.data_ptr(), workspace.numel() * workspace.element_size()),
               "fewbit_fwd_host")
    return y, packed


def fewbit_bwd_host(table: Table, packed: torch.Tensor, grad_out: torch.Tensor, grad_in: torch.Tensor,
                    workspace: torch.Tensor):
    """Backward half on host tensors; see ``fewbit_fwd_host``."""
    lib = load_library()
    _host_tensor(packed, "packed"), _host_tensor(grad_out, "grad_out"), _host_tensor(grad_in, "grad_in")
    _dev_tensor(workspace, "workspace")
    n = grad_out.numel()
    if grad_in.dtype != grad_out.dtype or grad_in.numel() != n or \
            packed.numel() * packed.element_size() < fewbit_packed_bytes(n, table.bits):
        raise ValueError("grad_in / packed do not match grad_out")
    with torch.cuda.device(workspace.device):
        _check(lib.fewbit_bwd_host(table.handle, packed.data_ptr(), grad_out.data_ptr(), grad_in.data_ptr(), n,
                                   _DTYPES[grad_out.dtype], workspace.data_ptr(),
                                   workspace.numel() * workspace.element_size()), "fewbit_bwd_host")
    return grad_in


def fewbit_static_max_elements() -> int:
    return int(load_library().fewbit_static_max_elements())


def fewbit_fwd_host_static(table: Table, x: torch.Tensor, y: torch.Tensor, packed: torch.Tensor,
                           stream: Optional[torch.cuda.Stream] = None, device=None):
    """Forward half on host tensors with no device allocation by anyone: the
    device staging area is a fixed array inside the library (at most
    ``fewbit_static_max_elements()`` elements per call).  For callers that
    cannot call cudaMalloc where they need the forward pass.  Blocks until the
    results are in ``y`` and ``packed``; calls must not overlap on one GPU."""
    lib = load_library()
    _host_tensor(x, "x"), _host_tensor(y, "y"), _host_tensor(packed, "packed")
    n = x.numel()
    if y.dtype != x.dtype or y.numel() != n or packed.numel() * packed.element_size() < fewbit_packed_bytes(n, table.bits):
        raise ValueError("y / packed do not match x")
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    with torch.cuda.device(device):
        _check(lib.fewbit_fwd_host_static(table.handle, x.data_ptr(), y.data_ptr(), packed.data_ptr(), n,
                                          _DTYPES[x.dtype], _stream_ptr(stream, device)), "fewbit_fwd_host_static")
    return y, packed
