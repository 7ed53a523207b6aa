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
