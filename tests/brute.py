"""Tiny-shape brute force used only to pin the oracle.

Contractions are done in exact rational arithmetic (every stored fp32 / bf16 value is a dyadic
rational) with a loop order different from the oracle's (output column outermost, contracted index
descending); transcendental steps use mpmath at 50 digits.  Pure Python: tiny shapes only.
"""
from fractions import Fraction

import mpmath as mp
import numpy as np

mp.mp.dps = 50


def to_fraction_array(a):
    """Stored tensor (float32 or uint16 bf16 patterns) -> nested list of Fractions (exact)."""
    if a.dtype == np.uint16:
        a = (a.astype(np.uint32) << np.uint32(16)).view(np.float32)
    flat = [Fraction(float(v)) for v in np.asarray(a, dtype=np.float64).ravel()]
    return np.array(flat, dtype=object).reshape(a.shape)


def gemm_nt(A, B):
    M, K = A.shape
    N, _ = B.shape
    V = np.empty((M, N), dtype=object)
    for n in range(N):
        for m in range(M):
            acc = Fraction(0)
            for k in reversed(range(K)):
                acc += A[m, k] * B[n, k]
            V[m, n] = acc
    return V


def conv2d_nhwc(x, w, stride, pad):
    NB, H, W, Cin = x.shape
    Cout, R, S, _ = w.shape
    OH = (H + 2 * pad - R) // stride + 1
    OW = (W + 2 * pad - S) // stride + 1
    V = np.empty((NB, OH, OW, Cout), dtype=object)
    # gather form over a zero-padded copy (the oracle skips taps instead)
    xp = np.empty((NB, H + 2 * pad, W + 2 * pad, Cin), dtype=object)
    xp[...] = Fraction(0)
    xp[:, pad:pad + H, pad:pad + W, :] = x
    for co in range(Cout):
        for b in range(NB):
            for ow in range(OW):
                for oh in range(OH):
                    acc = Fraction(0)
                    for ci in range(Cin):
                        for s in range(S):
                            for r in range(R):
                                acc += xp[b, oh * stride + r, ow * stride + s, ci] * w[co, r, s, ci]
                    V[b, oh, ow, co] = acc
    return V


def _mpf(v):
    if isinstance(v, Fraction):
        return mp.mpf(v.numerator) / mp.mpf(v.denominator)
    return mp.mpf(v)


def gelu_tanh(v):
    v = _mpf(v)
    c = mp.sqrt(2 / mp.pi)
    return v * (1 + mp.tanh(c * (v + mp.mpf("0.044715") * v ** 3))) / 2


def run_chain(chain, inputs):
    """Same contract as oracle.run_chain, returns float64 arrays; tiny shapes only."""
    fr = [to_fraction_array(a) for a in inputs]
    if chain.producer == "elementwise":
        V = fr[0].copy()
    elif chain.producer == "gemm_nt":
        V = gemm_nt(fr[0], fr[1])
    elif chain.producer == "conv2d_nchw":
        # channel-first storage is a relabelling of the same numbers: move the axes, then the channel-last sum
        V = conv2d_nhwc(fr[0].transpose(0, 2, 3, 1), fr[1].transpose(0, 2, 3, 1), chain.stride, chain.pad)
    else:
        V = conv2d_nhwc(fr[0], fr[1], chain.stride, chain.pad)
    shape = V.shape
    N = shape[-1]
    V = V.reshape(-1, N)
    V = np.array([[_mpf(v) for v in row] for row in V], dtype=object)
    for op in chain.ops:
        k = op[0]
        for m in range(V.shape[0]):
            for n in range(N):
                v = V[m, n]
                if k == "bias_n":
                    v = v + _mpf(fr[op[1]][n])
                elif k == "affine_n":
                    v = v * _mpf(fr[op[1]][n]) + _mpf(fr[op[2]][n])
                elif k == "relu":
                    v = v if v > 0 else mp.mpf(0)
                elif k == "gelu_tanh":
                    v = gelu_tanh(v)
                elif k == "scale":
                    v = v * mp.mpf(op[1])
                elif k == "clamp":
                    v = min(max(v, mp.mpf(op[1])), mp.mpf(op[2]))
                elif k == "add_tensor":
                    v = v + _mpf(fr[op[1]].reshape(-1, N)[m, n])
                else:
                    raise ValueError(k)
                V[m, n] = v
    out = {"main": np.array([[float(v) for v in row] for row in V]).reshape(shape)}
    if chain.reduce == "row_logsumexp":
        out["reduce"] = np.array([float(mp.log(mp.fsum([mp.exp(v) for v in row]))) for row in V])
    elif chain.reduce == "row_softmax":
        P = []
        for row in V:
            mx = max(row)
            e = [mp.exp(v - mx) for v in row]
            s = mp.fsum(e)
            P.append([float(x / s) for x in e])
        out["reduce"] = np.array(P).reshape(shape)
    elif chain.reduce in ("row_sum", "row_mean"):
        out["reduce"] = np.array([float(mp.fsum(list(row)) / (N if chain.reduce == "row_mean" else 1)) for row in V])
    elif chain.reduce == "row_max":
        out["reduce"] = np.array([float(max(row)) for row in V])
    elif chain.reduce == "global_avgpool":
        NB, OH, OW, C = shape
        V4 = V.reshape(NB, OH * OW, C)
        out["reduce"] = np.array([[float(mp.fsum(list(V4[b, :, c])) / (OH * OW)) for c in range(C)]
                                  for b in range(NB)])
    return out


def round_to_grid_fraction(v: Fraction, sig: int, emin_ulp: int) -> Fraction:
    """Nearest value with `sig` significant bits (ties to even), computed in exact rational arithmetic:
    an independent restatement of the 16-bit rounding (no floating point involved)."""
    if v == 0:
        return v
    a = abs(v)
    e = 0                       # find e with 2^(e-1) <= a < 2^e
    while Fraction(2) ** e <= a:
        e += 1
    while Fraction(2) ** (e - 1) > a:
        e -= 1
    ulp_e = max(e - sig, emin_ulp)
    scaled = a / Fraction(2) ** ulp_e
    q = scaled.numerator // scaled.denominator
    rem = scaled - q
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and q % 2 == 1):
        q += 1
    r = q * Fraction(2) ** ulp_e
    return r if v > 0 else -r
