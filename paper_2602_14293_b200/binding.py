"""ctypes binding with the same names as the C ABI (include/fc.h).

Argument marshalling only: every step of a chain runs inside the CUDA library.  torch is used for
device memory and streams.  There is no fallback: if the built library is missing, importing this
module fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import numpy as np
import torch

PKG = os.path.dirname(os.path.abspath(__file__))
# FC_LIBRARY selects another build of the same library (the bounds-checked libfc_debug.so); the default is the product
LIB_PATH = os.environ.get("FC_LIBRARY") or os.path.join(PKG, "libfc.so")

FC_F32, FC_BF16, FC_F16, FC_F8E4M3, FC_MXF8E4M3, FC_E8M0 = 0, 1, 2, 3, 4, 5
_PRODUCER = {"elementwise": 0, "gemm_nt": 1, "conv2d_nhwc": 2, "conv2d_nchw": 3}
_OPKIND = {"bias_n": 0, "affine_n": 1, "relu": 2, "gelu_tanh": 3, "scale": 4, "clamp": 5, "add_tensor": 6, "linear": 7}
_REDUCE = {"none": 0, "row_logsumexp": 1, "row_softmax": 2, "global_avgpool": 3, "row_sum": 4, "row_max": 5, "row_mean": 6, "maxpool_2x2": 7}
_DTYPE = {"f32": FC_F32, "bf16": FC_BF16, "f16": FC_F16, "f8e4m3": FC_F8E4M3, "mxf8e4m3": FC_MXF8E4M3}
FC_MAX_OPS = 12
FC_VERSION = 2


class fc_op(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("in0", ctypes.c_int32), ("in1", ctypes.c_int32),
                ("f0", ctypes.c_float), ("f1", ctypes.c_float)]


class fc_chain_spec(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("version", ctypes.c_uint32),
                ("producer", ctypes.c_int32), ("in_dtype", ctypes.c_int32),
                ("acc_dtype", ctypes.c_int32), ("out_dtype", ctypes.c_int32),
                ("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("batch", ctypes.c_int64), ("H", ctypes.c_int64), ("W", ctypes.c_int64),
                ("Cin", ctypes.c_int64), ("Cout", ctypes.c_int64), ("R", ctypes.c_int64),
                ("S", ctypes.c_int64), ("stride", ctypes.c_int64), ("pad", ctypes.c_int64),
                ("n_ops", ctypes.c_int32), ("ops", fc_op * FC_MAX_OPS),
                ("reduce", ctypes.c_int32), ("store_main", ctypes.c_int32)]


class fc_tensor(ctypes.Structure):
    _fields_ = [("ptr", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("rank", ctypes.c_int32),
                ("shape", ctypes.c_int64 * 4), ("stride", ctypes.c_int64 * 4)]


class FcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = lib().fc_status_string(status).decode()
        super().__init__(f"{where}: {name}: {fc_last_error()}")


_lib = None


def lib():
    """The loaded CUDA library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_14293_b200.build` "
                              "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        pt, ps = ctypes.POINTER(fc_tensor), ctypes.POINTER(fc_chain_spec)
        L.fc_run.argtypes = [ps, pt, ctypes.c_int, pt, ctypes.c_int, ctypes.c_void_p]
        L.fc_run.restype = ctypes.c_int
        L.fc_run_host.argtypes = [ps, pt, ctypes.c_int, pt, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        L.fc_run_host.restype = ctypes.c_int
        L.fc_staging_size.argtypes = [ps, pt, ctypes.c_int, pt, ctypes.c_int, ctypes.POINTER(ctypes.c_size_t)]
        L.fc_staging_size.restype = ctypes.c_int
        L.fc_run_softmax_static_scratch.argtypes = [ps, pt, ctypes.c_int, pt, ctypes.c_int, ctypes.c_void_p]
        L.fc_run_softmax_static_scratch.restype = ctypes.c_int
        L.fc_workspace_size.argtypes = [ps, ctypes.POINTER(ctypes.c_size_t)]
        L.fc_workspace_size.restype = ctypes.c_int
        L.fc_workspace_size_split.argtypes = [ps, ctypes.POINTER(ctypes.c_size_t)]
        L.fc_workspace_size_split.restype = ctypes.c_int
        L.fc_describe_plan.argtypes = [ps, ctypes.c_char_p, ctypes.c_size_t]
        L.fc_describe_plan.restype = ctypes.c_int
        L.fc_set_workspace.argtypes = [ctypes.c_void_p, ctypes.c_size_t]
        L.fc_set_workspace.restype = ctypes.c_int
        L.fc_get_async_status.argtypes = [ctypes.c_void_p]
        L.fc_get_async_status.restype = ctypes.c_int
        L.fc_launch_count.restype = ctypes.c_uint64
        L.fc_status_string.argtypes = [ctypes.c_int]
        L.fc_status_string.restype = ctypes.c_char_p
        L.fc_last_error.restype = ctypes.c_char_p
        L.fc_last_plan.restype = ctypes.c_char_p
        L.fc_version.restype = ctypes.c_int
        L.fc_testing_set.argtypes = [ctypes.c_int, ctypes.c_int]
        L.fc_testing_set.restype = None
        _lib = L
    return _lib


def fc_last_error() -> str:
    return lib().fc_last_error().decode()


def fc_last_plan() -> str:
    """Names of the kernel variants the last fc_run of this thread enqueued."""
    return lib().fc_last_plan().decode()


FC_TESTING_PANEL_STALL, FC_TESTING_SPLIT_STALL, FC_TESTING_BOUNDS_TRIP, FC_TESTING_TILE_WIDTH, FC_TESTING_POOL_FORM, FC_TESTING_BORDER_PASS = 0, 1, 2, 3, 4, 5


def fc_testing_set(which: int, value: int) -> None:
    """Testing switches of the library (see include/fc.h)."""
    lib().fc_testing_set(int(which), int(value))


def fc_version() -> int:
    return int(lib().fc_version())


def fc_launch_count() -> int:
    return int(lib().fc_launch_count())


def make_spec(chain) -> fc_chain_spec:
    """Build an fc_chain_spec from a declarative chain description (any object with the fields
    producer, in_dtype, out_dtype, M, N, K, batch, H, W, Cin, Cout, R, S, stride, pad, ops, reduce,
    store_main; ops are tuples such as ("bias_n", 2) or ("clamp", -1.0, 1.0))."""
    s = fc_chain_spec()
    s.struct_size = ctypes.sizeof(fc_chain_spec)
    s.version = FC_VERSION
    s.producer = _PRODUCER[chain.producer]
    s.in_dtype = _DTYPE[chain.in_dtype]
    s.acc_dtype = FC_F32
    s.out_dtype = _DTYPE[chain.out_dtype]
    for f in ("M", "N", "K", "batch", "H", "W", "Cin", "Cout", "R", "S", "stride", "pad"):
        setattr(s, f, int(getattr(chain, f)))
    s.n_ops = len(chain.ops)
    for i, op in enumerate(chain.ops):
        o = s.ops[i]
        o.kind = _OPKIND[op[0]]
        if op[0] in ("bias_n", "add_tensor", "linear"):
            o.in0 = int(op[1])
        elif op[0] == "affine_n":
            o.in0, o.in1 = int(op[1]), int(op[2])
        elif op[0] == "scale":
            o.f0 = float(op[1])
        elif op[0] == "clamp":
            o.f0, o.f1 = float(op[1]), float(op[2])
    s.reduce = _REDUCE[chain.reduce]
    s.store_main = 1 if chain.store_main else 0
    return s


def _tensor_struct(t: torch.Tensor) -> fc_tensor:
    ft = fc_tensor()
    ft.ptr = t.data_ptr()
    if t.dtype == torch.float32:
        ft.dtype = FC_F32
    elif t.dtype == torch.bfloat16:
        ft.dtype = FC_BF16
    elif t.dtype == torch.float16:
        ft.dtype = FC_F16
    elif t.dtype == torch.float8_e4m3fn:
        ft.dtype = FC_F8E4M3
    elif t.dtype == torch.uint8:          # scale bytes of block-scaled operands
        ft.dtype = FC_E8M0
    else:
        raise TypeError(f"unsupported dtype {t.dtype}")
    if t.dim() > 4:
        raise ValueError("rank > 4")
    ft.rank = t.dim()
    for i in range(t.dim()):
        ft.shape[i] = t.shape[i]
        ft.stride[i] = t.stride(i)
    return ft


def _tensor_array(ts: Sequence[torch.Tensor]):
    arr = (fc_tensor * max(1, len(ts)))()
    for i, t in enumerate(ts):
        arr[i] = _tensor_struct(t)
    return arr


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check(status: int, where: str):
    if status != 0:
        raise FcError(status, where)


def fc_run(spec: fc_chain_spec, inputs: Sequence[torch.Tensor], outputs: Sequence[torch.Tensor], stream=None) -> None:
    """fc_run of the C ABI: device tensors in, device tensors out, enqueued on `stream`."""
    _check(lib().fc_run(ctypes.byref(spec), _tensor_array(inputs), len(inputs), _tensor_array(outputs), len(outputs),
                        _stream_handle(stream)), "fc_run")


class PreparedRun:
    """The marshalled arguments of one fc_run call, built once: `run()` is then a single C call
    (building the ctypes structures costs more than a small kernel's run time)."""

    def __init__(self, spec: fc_chain_spec, inputs: Sequence[torch.Tensor], outputs: Sequence[torch.Tensor], stream=None):
        self._keep = (spec, list(inputs), list(outputs))      # keeps the tensors alive
        self._spec = ctypes.byref(spec)
        self._in, self._n_in = _tensor_array(inputs), len(inputs)
        self._out, self._n_out = _tensor_array(outputs), len(outputs)
        self._stream = _stream_handle(stream)
        self._fn = lib().fc_run

    def run(self) -> None:
        st = self._fn(self._spec, self._in, self._n_in, self._out, self._n_out, self._stream)
        if st != 0:
            raise FcError(st, "fc_run")


def fc_run_softmax_static_scratch(spec: fc_chain_spec, inputs: Sequence[torch.Tensor], outputs: Sequence[torch.Tensor],
                                  stream=None) -> None:
    """GEMM + row softmax for callers that cannot allocate: same arguments as fc_run, scratch taken from
    the fixed array built into the library (no workspace to register, nothing allocated).  Calls that
    overlap on the GPU share that array and race; see include/fc.h for the size limit."""
    _check(lib().fc_run_softmax_static_scratch(ctypes.byref(spec), _tensor_array(inputs), len(inputs),
                                               _tensor_array(outputs), len(outputs), _stream_handle(stream)),
           "fc_run_softmax_static_scratch")


def fc_staging_size(spec, inputs, outputs) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().fc_staging_size(ctypes.byref(spec), _tensor_array(inputs), len(inputs), _tensor_array(outputs),
                                 len(outputs), ctypes.byref(n)), "fc_staging_size")
    return int(n.value)


def fc_run_host(spec, host_inputs: Sequence[torch.Tensor], host_outputs: Sequence[torch.Tensor],
                staging: torch.Tensor, stream=None) -> None:
    """fc_run_host of the C ABI: host (ideally pinned) tensors in and out, `staging` a device byte buffer."""
    _check(lib().fc_run_host(ctypes.byref(spec), _tensor_array(host_inputs), len(host_inputs),
                             _tensor_array(host_outputs), len(host_outputs), ctypes.c_void_p(staging.data_ptr()),
                             staging.numel() * staging.element_size(), _stream_handle(stream)), "fc_run_host")


def fc_workspace_size(spec) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().fc_workspace_size(ctypes.byref(spec), ctypes.byref(n)), "fc_workspace_size")
    return int(n.value)


def fc_workspace_size_split(spec) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().fc_workspace_size_split(ctypes.byref(spec), ctypes.byref(n)), "fc_workspace_size_split")
    return int(n.value)


def fc_describe_plan(spec) -> dict:
    """How fc_run would execute `spec` now, as a dict ({"kernel": ..., "split": ..., ...}; numbers as int)."""
    buf = ctypes.create_string_buffer(256)
    _check(lib().fc_describe_plan(ctypes.byref(spec), buf, len(buf)), "fc_describe_plan")
    out = {}
    for item in buf.value.decode().split():
        k, v = item.split("=")
        out[k] = int(v) if v.lstrip("-").isdigit() else v
    return out


def fc_set_workspace(buf: Optional[torch.Tensor]) -> None:
    """Register `buf` (a uint8 device tensor, kept alive here) as the current device's workspace; None removes it."""
    if buf is None:
        _check(lib().fc_set_workspace(None, 0), "fc_set_workspace")
        _workspace.pop(torch.cuda.current_device(), None)
    else:
        _check(lib().fc_set_workspace(ctypes.c_void_p(buf.data_ptr()), buf.numel() * buf.element_size()), "fc_set_workspace")
        _workspace[buf.device.index] = buf


def fc_get_async_status(stream=None) -> None:
    _check(lib().fc_get_async_status(_stream_handle(stream)), "fc_get_async_status")


# --------------------------------------------------------------------------- conveniences
_TORCH_DT = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}
_workspace = {}


def to_device(a: np.ndarray, device="cuda") -> torch.Tensor:
    """Stored numpy tensor (float32, float16, uint16 bf16, uint8 E4M3 bit patterns or int8-tagged E8M0 scale bytes)
    -> torch tensor on `device`."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).to(device)
    if a.dtype == np.uint8:
        return torch.from_numpy(a).view(torch.float8_e4m3fn).to(device)
    if a.dtype == np.int8:                # E8M0 scale bytes (the generator tags them int8): plain bytes on the device
        return torch.from_numpy(a.view(np.uint8)).to(device)
    return torch.from_numpy(a).to(device)


def output_tensors(chain, device="cuda", pinned=False) -> List[torch.Tensor]:
    """Allocate (uninitialised) output tensors for `chain`, in the ABI's output order."""
    if chain.producer in ("conv2d_nhwc", "conv2d_nchw"):
        OH = (chain.H + 2 * chain.pad - chain.R) // chain.stride + 1
        OW = (chain.W + 2 * chain.pad - chain.S) // chain.stride + 1
        main_shape = (chain.batch, OH, OW, chain.Cout)
    else:
        main_shape = (chain.M, getattr(chain, "N_out", chain.N))
    kw = dict(device=device, pin_memory=pinned) if device == "cpu" else dict(device=device)
    outs = []
    if chain.reduce == "row_softmax" or chain.store_main:
        outs.append(torch.empty(main_shape, dtype=_TORCH_DT[chain.out_dtype], **kw))
    if chain.reduce in ("row_logsumexp", "row_sum", "row_max", "row_mean"):
        outs.append(torch.empty((chain.M,), dtype=torch.float32, **kw))
    elif chain.reduce == "global_avgpool":
        outs.append(torch.empty((chain.batch, chain.Cout), dtype=torch.float32, **kw))
    elif chain.reduce == "maxpool_2x2":
        dt = _TORCH_DT[chain.out_dtype] if chain.out_dtype in ("bf16", "f16") else torch.float32   # (as the library stores it)
        outs.append(torch.empty((chain.batch, OH // 2, OW // 2, chain.Cout), dtype=dt, **kw))
    return outs


def ensure_workspace(spec) -> None:
    """Register a torch-owned workspace large enough for `spec` (split tiles included) on the current device."""
    need = max(fc_workspace_size(spec), fc_workspace_size_split(spec))
    if need == 0:
        return
    dev = torch.cuda.current_device()
    cur = _workspace.get(dev)
    if cur is None or cur.numel() < need:
        cur = torch.empty(need, dtype=torch.uint8, device=f"cuda:{dev}")
        _workspace[dev] = cur
        fc_set_workspace(cur)


def run_chain(chain, inputs: Sequence[torch.Tensor], outputs: Optional[Sequence[torch.Tensor]] = None, stream=None):
    """Run `chain` on device tensors; allocates the outputs (torch) unless given.  Returns them."""
    spec = make_spec(chain)
    if outputs is None:
        outputs = output_tensors(chain, device=inputs[0].device)
    ensure_workspace(spec)
    fc_run(spec, inputs, outputs, stream)
    return list(outputs)


def run_chain_host(chain, host_inputs, host_outputs, staging, stream=None):
    spec = make_spec(chain)
    ensure_workspace(spec)
    fc_run_host(spec, host_inputs, host_outputs, staging, stream)
    return list(host_outputs)
