"""fp64 CPU oracle for fused operator chains (Python front of ``fc_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Imported by ``tests/``, by the smoke check and by the benchmark's
``cpu_baseline`` / ``--impl reference`` legs; the library's product path never touches it, and it
imports nothing from the CUDA package.

``run_chain(chain, inputs)`` evaluates a declarative chain (see ``fc_inputs.workloads.Chain``) as
the plain unfused definition: widen the stored inputs exactly to double, run the producer
(identity / GEMM NT / NHWC cross-correlation), apply the epilogue ops in the listed order, then the
reduction.  Nothing is rounded in between; outputs are float64 arrays.  Each step is one call into
the C file, whose header lists the passages it follows and the pins that check it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, List, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fc_oracle.c")
_LIB = os.path.join(_HERE, "libfc_oracle.so")
_lib = None

_i64 = ctypes.c_int64
_pd = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP, no fast-math). Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _p(a: np.ndarray):
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_pd)


def widen(a: np.ndarray) -> np.ndarray:
    """Stored tensor (float32, float16, uint16 bf16 patterns, uint8 E4M3 patterns, or int8-tagged E8M0 scale
    bytes) -> float64, exactly."""
    a = np.ascontiguousarray(a)
    out = np.empty(a.shape, dtype=np.float64)
    if a.dtype == np.int8:      # E8M0 scale bytes (the generator tags them with this dtype)
        lib().orc_widen_e8m0(a.ctypes.data_as(ctypes.c_void_p), _i64(a.size), _p(out))
    elif a.dtype == np.uint8:
        lib().orc_widen_f8e4m3(a.ctypes.data_as(ctypes.c_void_p), _i64(a.size), _p(out))
    elif a.dtype == np.uint16:
        lib().orc_widen_bf16(a.ctypes.data_as(ctypes.c_void_p), _i64(a.size), _p(out))
    elif a.dtype == np.float16:
        lib().orc_widen_f16(a.ctypes.data_as(ctypes.c_void_p), _i64(a.size), _p(out))
    elif a.dtype == np.float32:
        lib().orc_widen_f32(a.ctypes.data_as(ctypes.c_void_p), _i64(a.size), _p(out))
    elif a.dtype == np.float64:
        out[...] = a
    else:
        raise TypeError(a.dtype)
    return out


def gemm_nt(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    M, K = A.shape
    N, K2 = B.shape
    assert K == K2
    V = np.empty((M, N), dtype=np.float64)
    lib().orc_gemm_nt(_p(A), _p(B), _i64(M), _i64(N), _i64(K), _p(V))
    return V


def gemm_nt_mx(A: np.ndarray, B: np.ndarray, SA: np.ndarray, SB: np.ndarray) -> np.ndarray:
    """Block-scaled contraction: SA [M, K/32], SB [N, K/32] are the widened per-block scales."""
    M, K = A.shape
    N, K2 = B.shape
    assert K == K2 and K % 32 == 0 and SA.shape == (M, K // 32) and SB.shape == (N, K // 32)
    V = np.empty((M, N), dtype=np.float64)
    lib().orc_gemm_nt_mx(_p(A), _p(B), _p(SA), _p(SB), _i64(M), _i64(N), _i64(K), _p(V))
    return V


def conv2d_nhwc(x: np.ndarray, w: np.ndarray, stride: int, pad: int) -> np.ndarray:
    NB, H, W, Cin = x.shape
    Cout, R, S, Cin2 = w.shape
    assert Cin == Cin2
    OH = (H + 2 * pad - R) // stride + 1
    OW = (W + 2 * pad - S) // stride + 1
    V = np.empty((NB, OH, OW, Cout), dtype=np.float64)
    lib().orc_conv2d_nhwc(_p(x), _p(w), _i64(NB), _i64(H), _i64(W), _i64(Cin), _i64(Cout),
                          _i64(R), _i64(S), _i64(stride), _i64(pad), _p(V))
    return V


def conv2d_nchw(x: np.ndarray, w: np.ndarray, stride: int, pad: int) -> np.ndarray:
    """Image [NB, Cin, H, W], weights [Cout, Cin, R, S]; returns V[NB, OH, OW, Cout] (channels last)."""
    NB, Cin, H, W = x.shape
    Cout, Cin2, R, S = w.shape
    assert Cin == Cin2
    OH = (H + 2 * pad - R) // stride + 1
    OW = (W + 2 * pad - S) // stride + 1
    V = np.empty((NB, OH, OW, Cout), dtype=np.float64)
    lib().orc_conv2d_nchw(_p(x), _p(w), _i64(NB), _i64(H), _i64(W), _i64(Cin), _i64(Cout),
                          _i64(R), _i64(S), _i64(stride), _i64(pad), _p(V))
    return V


def apply_op(V: np.ndarray, op: tuple, inputs64: Sequence[np.ndarray]) -> None:
    """Apply one epilogue op in place to V (viewed as [rows, N] with N the last axis)."""
    L = lib()
    N = V.shape[-1]
    rows = V.size // N
    kind = op[0]
    if kind == "bias_n":
        b = inputs64[op[1]]
        assert b.shape == (N,)
        L.orc_bias_n(_p(V), _i64(rows), _i64(N), _p(b))
    elif kind == "affine_n":
        g, b = inputs64[op[1]], inputs64[op[2]]
        assert g.shape == (N,) and b.shape == (N,)
        L.orc_affine_n(_p(V), _i64(rows), _i64(N), _p(g), _p(b))
    elif kind == "relu":
        L.orc_relu(_p(V), _i64(V.size))
    elif kind == "gelu_tanh":
        L.orc_gelu_tanh(_p(V), _i64(V.size))
    elif kind == "scale":
        L.orc_scale(_p(V), _i64(V.size), ctypes.c_double(op[1]))
    elif kind == "clamp":
        L.orc_clamp(_p(V), _i64(V.size), ctypes.c_double(op[1]), ctypes.c_double(op[2]))
    elif kind == "add_tensor":
        t = inputs64[op[1]]
        assert t.shape == V.shape
        L.orc_add_tensor(_p(V), _i64(V.size), _p(t))
    else:
        raise ValueError(kind)


def row_logsumexp(V: np.ndarray) -> np.ndarray:
    rows, N = V.shape
    out = np.empty((rows,), dtype=np.float64)
    lib().orc_row_logsumexp(_p(V), _i64(rows), _i64(N), _p(out))
    return out


def row_softmax(V: np.ndarray) -> np.ndarray:
    rows, N = V.shape
    P = np.empty_like(V)
    lib().orc_row_softmax(_p(V), _i64(rows), _i64(N), _p(P))
    return P


def row_sum(V: np.ndarray) -> np.ndarray:
    rows, N = V.shape
    out = np.empty((rows,), dtype=np.float64)
    lib().orc_row_sum(_p(V), _i64(rows), _i64(N), _p(out))
    return out


def row_max(V: np.ndarray) -> np.ndarray:
    rows, N = V.shape
    out = np.empty((rows,), dtype=np.float64)
    lib().orc_row_max(_p(V), _i64(rows), _i64(N), _p(out))
    return out


def global_avgpool(V: np.ndarray) -> np.ndarray:
    NB, OH, OW, C = V.shape
    out = np.empty((NB, C), dtype=np.float64)
    lib().orc_global_avgpool(_p(V), _i64(NB), _i64(OH * OW), _i64(C), _p(out))
    return out


def round_to(V: np.ndarray, dtype: str) -> np.ndarray:
    """A copy of V rounded (nearest, ties to even) onto the grid of the storage type ('f32': unchanged)."""
    out = np.ascontiguousarray(V, dtype=np.float64).copy()
    if dtype == "bf16":
        lib().orc_round_bf16(_p(out), _i64(out.size))
    elif dtype == "f16":
        lib().orc_round_f16(_p(out), _i64(out.size))
    elif dtype != "f32":
        raise ValueError(dtype)
    return out


def maxpool_2x2(V: np.ndarray) -> np.ndarray:
    NB, OH, OW, C = V.shape
    out = np.empty((NB, OH // 2, OW // 2, C), dtype=np.float64)
    lib().orc_maxpool_2x2(_p(V), _i64(NB), _i64(OH), _i64(OW), _i64(C), _p(out))
    return out


def run_chain(chain, inputs: List[np.ndarray]) -> Dict[str, np.ndarray]:
    """Evaluate ``chain`` on stored ``inputs``.  Returns {"main": f64 array, "reduce": f64 array}
    ("reduce" only when the chain has a reduction; "main" is always the pre-reduction tensor)."""
    x64 = [widen(a) for a in inputs]
    if chain.producer == "elementwise":
        V = x64[0].copy()
    elif chain.producer == "gemm_nt" and chain.in_dtype == "mxf8e4m3":
        V = gemm_nt_mx(x64[0], x64[1], x64[2], x64[3])     # inputs 2, 3: the per-block scales of A and B
    elif chain.producer == "gemm_nt":
        V = gemm_nt(x64[0], x64[1])
    elif chain.producer == "conv2d_nhwc":
        V = conv2d_nhwc(x64[0], x64[1], chain.stride, chain.pad)
    elif chain.producer == "conv2d_nchw":
        V = conv2d_nchw(x64[0], x64[1], chain.stride, chain.pad)
    else:
        raise ValueError(chain.producer)
    for op in chain.ops:
        if op[0] == "linear":
            # the next contraction takes the activation as stored in the chain's 16-bit type
            V = gemm_nt(round_to(V, chain.in_dtype), x64[op[1]])
        else:
            apply_op(V, op, x64)
    out = {"main": V}
    if chain.reduce == "row_logsumexp":
        out["reduce"] = row_logsumexp(V.reshape(-1, V.shape[-1]))
    elif chain.reduce == "row_softmax":
        out["reduce"] = row_softmax(V.reshape(-1, V.shape[-1]))
    elif chain.reduce == "global_avgpool":
        out["reduce"] = global_avgpool(V)
    elif chain.reduce == "maxpool_2x2":
        out["reduce"] = maxpool_2x2(V)
    elif chain.reduce == "row_sum":
        out["reduce"] = row_sum(V.reshape(-1, V.shape[-1]))
    elif chain.reduce == "row_max":
        out["reduce"] = row_max(V.reshape(-1, V.shape[-1]))
    elif chain.reduce == "row_mean":
        out["reduce"] = row_sum(V.reshape(-1, V.shape[-1])) / V.shape[-1]
    elif chain.reduce != "none":
        raise ValueError(chain.reduce)
    return out
