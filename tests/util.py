"""Helpers of the parity tests: comparison criteria, sampling, NaN-poisoned outputs."""
import numpy as np
import torch

from fc_inputs import rng


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Device / host tensor -> float64 numpy, exact widening."""
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        bits = t.view(torch.int16).numpy().view(np.uint16)
        return rng.bf16_bits_to_f32(bits).astype(np.float64)
    return t.numpy().astype(np.float64)


def check_f32(got: np.ndarray, ref: np.ndarray, what=""):
    """fp32 outputs: every element within 1e-4 * (1 + |ref|)."""
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite values in the output"
    err = np.abs(got - ref)
    bound = 1e-4 * (1.0 + np.abs(ref))
    worst = float((err / bound).max())
    assert worst <= 1.0, f"{what}: max |err| / (1e-4 (1+|ref|)) = {worst:.3f} at {np.unravel_index((err / bound).argmax(), err.shape)}"
    return worst


def check_bf16(got: np.ndarray, ref: np.ndarray, what=""):
    """bf16 outputs with fp32 accumulation: max relative error <= 2e-2 and mean absolute error <= 2e-3.
    Relative error of element i is |g - r| / max(|r|, 0.1 rms(ref)): the floor keeps the measure
    meaningful where the reference passes through zero and scales with the output's magnitude."""
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite values in the output"
    err = np.abs(got - ref)
    floor = 0.1 * float(np.sqrt(np.mean(ref * ref)))
    rel = err / np.maximum(np.abs(ref), max(floor, 1e-30))
    mx, mean_abs = float(rel.max()), float(err.mean())
    assert mx <= 2e-2, f"{what}: max rel err {mx:.4g} at {np.unravel_index(rel.argmax(), rel.shape)}"
    # a mean over a handful of elements is just one element's bf16 rounding (up to 2^-9 |ref|):
    # below 256 elements the bound scales with the largest magnitude present
    mean_bound = 2e-3 if ref.size >= 256 else 2e-3 * max(1.0, float(np.abs(ref).max()))
    assert mean_abs <= mean_bound, f"{what}: mean abs err {mean_abs:.4g}"
    return mx, mean_abs


def check_f16(got: np.ndarray, ref: np.ndarray, what=""):
    """fp16 outputs (the benchmark states no tolerance for them): one round-to-nearest to an 11-bit
    significand is 2^-11 = 4.9e-4 relative, so max relative error <= 2e-3 (same floor as for bf16)
    and mean absolute error <= 2.5e-4, i.e. the bf16 bounds tightened by the 8x finer grid."""
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite values in the output"
    err = np.abs(got - ref)
    floor = 0.1 * float(np.sqrt(np.mean(ref * ref)))
    rel = err / np.maximum(np.abs(ref), max(floor, 1e-30))
    mx, mean_abs = float(rel.max()), float(err.mean())
    assert mx <= 2e-3, f"{what}: max rel err {mx:.4g} at {np.unravel_index(rel.argmax(), rel.shape)}"
    mean_bound = 2.5e-4 if ref.size >= 256 else 2.5e-4 * max(1.0, float(np.abs(ref).max()))
    assert mean_abs <= mean_bound, f"{what}: mean abs err {mean_abs:.4g}"
    return mx, mean_abs


def check(got_t: torch.Tensor, ref: np.ndarray, what=""):
    got = to_f64(got_t)
    if got_t.dtype == torch.bfloat16:
        return check_bf16(got, ref, what)
    if got_t.dtype == torch.float16:
        return check_f16(got, ref, what)
    return check_f32(got, ref, what)


def poison_(ts):
    """Fill outputs with NaN patterns so that an element the kernel never writes fails the check."""
    for t in ts:
        t.fill_(float("nan"))
    return ts


def check_chained(got_t: torch.Tensor, ref: np.ndarray, allowance: np.ndarray, what=""):
    """Outputs of chained linear layers.  Between layers an activation is rounded to the 16-bit grid; where
    its fp32 value lies within accumulation error of a rounding boundary, the kernel and the fp64 oracle may
    legitimately pick neighbouring grid points (so would an unfused sequence).  `allowance[m][n]` bounds what
    two such picks per hidden layer can do to output (m, n).  Criteria: the usual per-element bound of the
    output type, widened by the allowance; at most 0.5 % of the elements may need the allowance at all; and
    the mean absolute error keeps its usual bound (a systematic error cannot hide behind rare flips)."""
    got = to_f64(got_t)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite values in the output"
    err = np.abs(got - ref)
    floor = 0.1 * float(np.sqrt(np.mean(ref * ref)))
    if got_t.dtype == torch.float32:
        base, mean_bound = 1e-4 * (1.0 + np.abs(ref)), None
    else:
        f16 = got_t.dtype == torch.float16
        base = (2e-3 if f16 else 2e-2) * np.maximum(np.abs(ref), max(floor, 1e-30))
        mean_bound = (2.5e-4 if f16 else 2e-3) * (1.0 if ref.size >= 256 else max(1.0, float(np.abs(ref).max())))
    over = err > base
    assert over.mean() <= 5e-3, f"{what}: {over.mean():.4%} of the elements exceed the plain bound"
    worst = float((err / (base + allowance)).max())
    assert worst <= 1.0, f"{what}: |err| / (bound + flip allowance) = {worst:.3f} at {np.unravel_index((err / (base + allowance)).argmax(), err.shape)}"
    if mean_bound is not None:
        assert float(err.mean()) <= mean_bound, f"{what}: mean abs err {float(err.mean()):.4g}"
    return float(over.mean()), worst


def flip_allowance(orc, ch, ins):
    """What two neighbouring-grid-point picks per hidden layer can do to each output: for hidden layer l with
    activations h (before rounding) and the remaining layers' weights W_{l+1} .. W_L, a pick moves h[m][k] by
    one grid step ulp(h[m][k]) and output (m, n) by at most (|W_L| ... |W_{l+1}|)[n][k] ulp(h[m][k]) times the
    activations' Lipschitz constant (1 for ReLU, below 1.13 for tanh-GELU)."""
    x = [orc.widen(a) for a in ins]
    sig = 8 if ch.in_dtype == "bf16" else 11
    V = orc.gemm_nt(x[0], x[1])
    hidden, weights = [], []
    for op in ch.ops:
        if op[0] == "linear":
            hidden.append(V.copy())
            weights.append(x[op[1]])
            V = orc.gemm_nt(orc.round_to(V, ch.in_dtype), x[op[1]])
        else:
            orc.apply_op(V, op, x)
    allowance = np.zeros_like(V)
    for l, h in enumerate(hidden):
        J = np.abs(weights[-1])
        for w in reversed(weights[l:-1]):
            J = 1.13 * (J @ np.abs(w))                      # [N_out, width of layer l]
        with np.errstate(divide="ignore"):
            ulp = np.where(h != 0, np.exp2(np.floor(np.log2(np.abs(h) + 1e-300)) - (sig - 1)), 0.0)
        allowance += 2.0 * 1.13 * np.max(ulp[:, None, :] * J[None, :, :], axis=2)
    return allowance
