"""Parity of the CUDA path with the CPU oracle, element by element, through the C ABI.

Tolerances (written here, as the benchmark states them): fp32 outputs |err| <= 1e-4 (1 + |ref|)
for every element; bf16 outputs max relative error <= 2e-2 and mean absolute error <= 2e-3.
Integer-valued contractions must agree bit for bit.  Outputs are NaN-poisoned before every run.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

from fc_inputs import rng, workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fc():
    import __graft_entry__ as entry
    entry.build()
    import paper_2602_14293_b200 as fc
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    torch.cuda.set_device(0)
    return fc


def run_and_check(fc, orc, ch, seed=0, ins=None, tag=""):
    if ins is None:
        ins = wl.make_inputs(ch, seed)
    ref = orc.run_chain(ch, ins)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    before = fc.fc_launch_count()
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    assert fc.fc_launch_count() > before, "no kernel of the library was launched"
    names = [r for r, _, _ in wl.output_shapes(ch)]
    res = {}
    for name, t in zip(names, outs):
        res[name] = util.check(t, ref[name], f"{ch.name}{tag} seed {seed}: {name}")
    return outs, ref, res


def run_without_workspace(fc, orc, ch, seed=0, ins=None):
    """The same through fc_run with no workspace registered: the forms that need no scratch (an eight-channel image
    with padding then takes eight filter taps per k-block instead of the bordered copy + filter rows)."""
    if ins is None:
        ins = wl.make_inputs(ch, seed)
    ref = orc.run_chain(ch, ins) if orc is not None else None
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.binding.fc_set_workspace(None)
    fc.binding.fc_run(fc.make_spec(ch), [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    if ref is not None:
        for (name, _, _), t in zip(wl.output_shapes(ch), outs):
            util.check(t, ref[name], f"{ch.name} without workspace, seed {seed}: {name}")
    return outs


# ------------------------------------------------------------------ C1: strict fp32 GEMM + bias + ReLU
@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("variant", ["std", "var"])
def test_c1_gemm_f32(fc, orc, seed, variant):
    run_and_check(fc, orc, wl.gemm_bias_relu_f32(256, 256, 256, variant), seed)


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (33, 65, 70), (100, 37, 129), (257, 31, 32)])
def test_gemm_f32_ragged(fc, orc, M, N, K):
    run_and_check(fc, orc, wl.gemm_bias_relu_f32(M, N, K, "var"), 3)


@pytest.mark.parametrize("M,N,K,plan", [(1500, 1100, 260, "big"), (1300, 1290, 131, "big"), (2048, 1024, 64, "big"), (900, 1800, 16, "big"),
                                        (1500, 1100, 7, "big"), (700, 900, 260, "mid"), (1025, 600, 131, "mid"), (520, 1030, 7, "mid"),
                                        (33, 16300, 72, "mid")])
def test_gemm_f32_large_register_tiled(fc, orc, M, N, K, plan):
    """Larger strict-fp32 GEMMs run register-tiled: 128 x 128 tiles (8 x 8 outputs per thread) from 96 such tiles
    on, 64 x 64 tiles (4 x 4) below.  Ragged edges in all three extents, K off the 16-byte grid (scalar loads),
    N off it (scalar stores)."""
    run_and_check(fc, orc, wl.gemm_bias_relu_f32(M, N, K, "var"), 5)
    assert fc.fc_last_plan() == "gemm_f32_" + plan


@pytest.mark.parametrize("M,N,K", [(2048, 2048, 2048), (1100, 1300, 516), (700, 4003, 260), (4100, 300, 1024)])
@pytest.mark.parametrize("variant", ["std", "var"])
def test_gemm_f32_on_tensor_cores(fc, orc, M, N, K, variant):
    """fp32 GEMMs of 2^29 multiply-adds and more, K a multiple of 4, with a workspace: two layout launches cut every
    operand into the part a tf32 multiplication reads and the rest, and the tensor-core kernel contracts
    [A_lo | A_hi | A_hi] with [B_hi | B_lo | B_hi] in fp32 accumulators.  Same fp32 tolerance as the FMA kernels; ragged
    extents, rows of the output off 16-byte boundaries."""
    ch = wl.gemm_bias_relu_f32(M, N, K, variant)
    run_and_check(fc, orc, ch, 6)
    assert fc.fc_last_plan().startswith("split_tf32 split_tf32 gemm_tc_mode7_bn")
    assert fc.binding.fc_describe_plan(fc.make_spec(ch))["kernel"] == "gemm_tc"


@pytest.mark.parametrize("ops", [
    (("affine_n", 2, 3), ("gelu_tanh",), ("scale", 0.5), ("clamp", -1.0, 1.0), ("add_tensor", 4)),   # the fused packed form
    (("relu",), ("bias_n", 2), ("scale", 2.0), ("add_tensor", 4), ("clamp", -0.5, 3.0)),                # interpreted op by op
    (),
])
def test_gemm_f32_on_tensor_cores_op_lists(fc, orc, ops):
    """The tensor-core form of the fp32 GEMM shares the 16-bit GEMM's epilogue: fp32 vectors and an fp32 residual,
    fused and interpreted op lists, an empty one; ragged extents at the smallest size that takes this path."""
    M, N, K = 1030, 1100, 512
    rec = (("A", "f32", (M, K), "normal", 0.0, K ** -0.25), ("B", "f32", (N, K), "normal", 0.0, K ** -0.25),
           ("v0", "f32", (N,), "uniform", -0.1, 0.1), ("v1", "f32", (N,), "normal", 1.0, 0.1), ("t", "f32", (M, N), "normal", 0.0, 1.0))
    ch = wl.Chain("gemm_f32_ops", "gemm_nt", "f32", "f32", M=M, N=N, K=K, ops=ops, input_recipe=rec)
    run_and_check(fc, orc, ch, 7)
    assert "gemm_tc_mode7" in fc.fc_last_plan()


def test_gemm_f32_on_tensor_cores_non_finite_operands(fc, orc):
    """Infinities and NaNs among the operands of the tensor-core fp32 GEMM: every output is an infinity of the right
    sign, a NaN, or a finite value within tolerance exactly where the fp64 contraction says so (the non-finite values
    sit at different k, see the split kernel)."""
    M, N, K = 1030, 1100, 512
    ch = wl.Chain("gemm_f32_nonfinite", "gemm_nt", "f32", "f32", M=M, N=N, K=K, ops=(),
                  input_recipe=(("A", "f32", (M, K), "normal", 0.0, K ** -0.25), ("B", "f32", (N, K), "normal", 0.0, K ** -0.25)))
    A, B = (np.array(t, dtype=np.float32) for t in wl.make_inputs(ch, 8))
    A[5, 7] = np.inf; A[9, 100] = np.nan; A[700, 300] = -np.inf
    B[11, 3] = -np.inf; B[900, 44] = np.inf; B[17, 7] = 0.25       # (exactly representable in tf32: its lo part is zero)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(A), fc.to_device(B)], outs)
    fc.fc_get_async_status()
    assert "gemm_tc_mode7" in fc.fc_last_plan()
    got = outs[0].cpu().numpy().astype(np.float64)
    with np.errstate(invalid="ignore", over="ignore"):
        ref = A.astype(np.float64) @ B.astype(np.float64).T
    assert (np.isnan(got) == np.isnan(ref)).all()
    assert (np.isposinf(got) == np.isposinf(ref)).all() and (np.isneginf(got) == np.isneginf(ref)).all()
    fin = np.isfinite(ref)
    assert fin.sum() > 0.99 * ref.size
    assert (np.abs(got[fin] - ref[fin]) <= 1e-4 * (1.0 + np.abs(ref[fin]))).all()


def test_gemm_f32_large_without_workspace_or_alignment_stays_on_the_alus(fc, orc):
    """The same sizes without a registered workspace, or with K off the 16-byte grid, take the fp32-FMA kernel."""
    ch = wl.gemm_bias_relu_f32(1100, 1300, 516, "var")
    ins = wl.make_inputs(ch, 6)
    ref = orc.run_chain(ch, ins)
    spec = fc.make_spec(ch)
    assert fc.binding.fc_workspace_size(spec) > 0
    fc.binding.fc_set_workspace(None)
    fc.binding._workspace.clear()
    assert fc.binding.fc_describe_plan(spec)["kernel"] == "gemm_f32"
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.fc_run(spec, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    assert fc.fc_last_plan() == "gemm_f32_big"
    util.check(outs[0], ref["main"], "fp32 GEMM without workspace")
    ch2 = wl.gemm_bias_relu_f32(1100, 1300, 514, "var")
    assert fc.binding.fc_workspace_size(fc.make_spec(ch2)) == 0
    run_and_check(fc, orc, ch2, 6)
    assert fc.fc_last_plan() == "gemm_f32_big"


# ------------------------------------------------------------------ kernel (a): elementwise + logsumexp
@pytest.mark.parametrize("M,N", [(1, 1), (3, 8), (5, 1000), (7, 4097), (33, 2048), (64, 4096), (9, 12345)])
def test_elementwise_lse_shapes(fc, orc, M, N):
    run_and_check(fc, orc, wl.affine_gelu_residual_lse(M, N), 1)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_c2_reduced_rows(fc, orc, seed):
    run_and_check(fc, orc, wl.affine_gelu_residual_lse(1024, 4096), seed)


def test_elementwise_f32_and_other_op_lists(fc, orc):
    base = wl.affine_gelu_residual_lse(37, 515)
    rec32 = tuple((t, "f32", s, d, a, b) for t, _, s, d, a, b in base.input_recipe)
    # fp32 storage in and out, no reduction
    run_and_check(fc, orc, replace(base, in_dtype="f32", out_dtype="f32", reduce="none", input_recipe=rec32), 2)
    # logsumexp only (main output not stored)
    run_and_check(fc, orc, replace(base, store_main=False), 2)
    # bias -> relu -> scale -> clamp on bf16, no reduction
    ch = replace(base, ops=(("bias_n", 1), ("relu",), ("scale", 0.5), ("clamp", -0.25, 0.75), ("add_tensor", 3)), reduce="none")
    run_and_check(fc, orc, ch, 2)
    # no ops at all: a copy with logsumexp
    run_and_check(fc, orc, replace(base, ops=()), 2)


@pytest.mark.parametrize("M,N", [(1, 1), (1000, 8), (777, 64), (301, 72), (123, 200), (50, 255), (3000, 13), (9, 256), (4, 3000)])
@pytest.mark.parametrize("dt", ["bf16", "f32"])
def test_elementwise_without_reduction_walks_the_tensor_flat(fc, orc, M, N, dt):
    """No reduction: the grid walks the chunks of the whole tensor, whatever the row length (narrow rows would
    otherwise idle most of a CTA); per-column vectors and the residual must still line up with the columns,
    also when a row is no multiple of eight columns."""
    base = wl.affine_gelu_residual_lse(M, N)
    if dt == "f32":
        base = replace(base, in_dtype="f32", out_dtype="f32", input_recipe=tuple((t, "f32", s, d, a, b) for t, _, s, d, a, b in base.input_recipe))
    run_and_check(fc, orc, replace(base, reduce="none"), 6)
    run_and_check(fc, orc, replace(base, reduce="none", ops=(("bias_n", 2), ("relu",), ("add_tensor", 3))), 6)
    run_and_check(fc, orc, wl.cast(M, N, "f32", "bf16" if dt == "bf16" else "f16"), 6)


@pytest.mark.parametrize("M,N", [(1, 1), (3, 8), (5, 1000), (7, 4097), (33, 2048), (64, 4096), (9, 12345), (300, 64)])
@pytest.mark.parametrize("dt", ["bf16", "f32", "f16"])
def test_elementwise_row_softmax(fc, orc, M, N, dt):
    ch = wl.scale_add_softmax(M, N, dtype=dt)
    outs, ref, _ = run_and_check(fc, orc, ch, 8)
    sums = util.to_f64(outs[0]).sum(axis=1)
    np.testing.assert_allclose(sums, 1.0, atol=2e-2 if dt == "bf16" else 2e-3)


def test_elementwise_row_softmax_other_op_lists_and_extremes(fc, orc):
    base = wl.scale_add_softmax(40, 777)
    # no ops; affine -> GELU in front; a dominant logit per row and rows shifted by +-1e4 (fp32 storage)
    run_and_check(fc, orc, replace(base, ops=()), 1)
    aff = wl.affine_gelu_residual_lse(40, 777)
    run_and_check(fc, orc, replace(aff, reduce="row_softmax", store_main=False), 1)
    ch32 = wl.scale_add_softmax(16, 515, scale=1.0, dtype="f32")
    ins = wl.make_inputs(ch32, 2)
    ins[0][np.arange(16), np.arange(16) * 3] += 60.0
    ins[0][::2] += 1.0e4
    ins[0][1::2] -= 1.0e4
    outs, ref, _ = run_and_check(fc, orc, ch32, ins=ins)
    assert (util.to_f64(outs[0]).argmax(1) == np.arange(16) * 3).all()


@pytest.mark.parametrize("N,dt", [(1000, "bf16"), (4096, "bf16"), (515, "f32"), (20000, "bf16")])
@pytest.mark.parametrize("red", ["row_softmax", "row_logsumexp"])
def test_elementwise_softmax_and_logsumexp_with_minus_infinity_masks(fc, orc, N, dt, red):
    """An additive mask of 0 / -inf (causal: row i keeps columns <= 37 i + 5; plus a row that keeps a single
    column in the middle and rows masked on the left): masked entries get probability exactly 0, whole
    stretches of -inf at the start, in the middle or at the end of a lane's columns leave the rest intact."""
    M = 24
    ch = replace(wl.scale_add_softmax(M, N, dtype=dt), reduce=red, store_main=False)   # (a stored main output would hold the -inf itself)
    ins = wl.make_inputs(ch, 12)
    keep = np.arange(N)[None, :] <= (37 * np.arange(M)[:, None] + 5)
    keep[3] = False; keep[3, N // 2] = True
    keep[5] = np.arange(N) >= N - 9
    keep[7] = (np.arange(N) // 64) % 2 == 1
    mask = np.where(keep, 0.0, -np.inf).astype(np.float32)
    ins[1] = rng.store(mask, dt)
    outs, ref, _ = run_and_check(fc, orc, ch, ins=ins)
    if red == "row_softmax":
        got = util.to_f64(outs[0])
        assert (got[~keep] == 0.0).all()
        np.testing.assert_allclose(got.sum(1), 1.0, atol=2e-2 if dt == "bf16" else 1e-4)


@pytest.mark.parametrize("red", ["row_softmax", "row_logsumexp"])
def test_gemm_softmax_and_logsumexp_with_minus_infinity_mask(fc, orc, red):
    """Scores = A B^T * scale + mask with a causal 0 / -inf mask (the attention-score chain): whole tiles, half
    rows of a tile and single columns of -inf; masked probabilities are exactly 0."""
    M, N, K = 300, 1000, 136
    base = wl.gemm_softmax(M, N, K, "var")
    rec = base.input_recipe + (("mask", "bf16", (M, N), "normal", 0.0, 1.0),)
    ch = replace(base, ops=(("scale", 0.5), ("add_tensor", 2)), reduce=red, store_main=False, input_recipe=rec)
    ins = wl.make_inputs(ch, 4)
    keep = np.arange(N)[None, :] <= (3 * np.arange(M)[:, None] + 2)
    keep[7] = False; keep[7, 600] = True
    keep[9] = np.arange(N) >= 900
    ins[2] = rng.store(np.where(keep, 0.0, -np.inf).astype(np.float32), "bf16")
    outs, ref, _ = run_and_check(fc, orc, ch, ins=ins)
    if red == "row_softmax":
        got = util.to_f64(outs[0])
        assert (got[~keep] == 0.0).all()
        np.testing.assert_allclose(got.sum(1), 1.0, atol=2e-2)


@pytest.mark.parametrize("ops", [
    (("bias_n", 2), ("relu",), ("scale", 0.5), ("clamp", -0.25, 0.75), ("add_tensor", 3)),
    (("affine_n", 1, 2), ("gelu_tanh",), ("clamp", -0.5, 1.5)),
    (("gelu_tanh",), ("scale", 3.0)),
    (("scale", 0.5), ("bias_n", 1), ("scale", 2.0), ("clamp", -1.0, 1.0), ("add_tensor", 3)),
    (("clamp", -0.3, 0.3),),
])
@pytest.mark.parametrize("red", ["none", "row_logsumexp", "row_sum"])
@pytest.mark.parametrize("M,N,dt", [(37, 512, "bf16"), (64, 4096, "f16"), (5, 264, "bf16")])
def test_elementwise_scale_and_clamp_behind_the_activation(fc, orc, ops, red, M, N, dt):
    """Op lists [scale] [bias | affine] [relu | gelu] [scale] [clamp] [add tensor] take the row kernel (16-bit
    storage, N a multiple of 8); the residual is then added behind the clamp, not inside the activation."""
    base = wl.affine_gelu_residual_lse(M, N)
    if dt == "f16":
        base = _as_f16(base)
    run_and_check(fc, orc, replace(base, ops=ops, reduce=red, store_main=True), 13)


@pytest.mark.parametrize("M,N", [(5, 12288), (3, 50264), (9, 24584), (2, 100000)])
@pytest.mark.parametrize("dt", ["bf16", "f16"])
def test_elementwise_long_rows_take_a_cta_per_row(fc, orc, M, N, dt):
    """Rows from 12288 columns on (a vocabulary): a CTA per row, vectors read from their 16-bit originals.  Row
    logsumexp with and without the main output, row softmax (second pass from L2), sum / max / mean, and a
    -inf mask over most of a row."""
    base = wl.affine_gelu_residual_lse(M, N)
    sm = wl.scale_add_softmax(M, N)
    if dt == "f16":
        base, sm = _as_f16(base), _as_f16(sm)
    run_and_check(fc, orc, base, 3)
    run_and_check(fc, orc, replace(base, store_main=False, ops=(("bias_n", 2), ("relu",))), 3)
    # (probabilities below 6e-5 are fp16 subnormals: their storage rounding alone exceeds the fp16 tolerance)
    if dt == "bf16" or N <= 12288:
        run_and_check(fc, orc, sm, 3)
    for red in ("row_sum", "row_max", "row_mean"):
        run_and_check(fc, orc, replace(base, reduce=red, ops=(("scale", 0.5), ("bias_n", 1))), 3)
    ins = wl.make_inputs(sm, 5)
    keep = np.arange(N)[None, :] % 1000 < (np.arange(M)[:, None] + 1)
    ins[1] = rng.store(np.where(keep, 0.0, -np.inf).astype(np.float32), dt)
    outs, _, _ = run_and_check(fc, orc, sm, ins=ins)
    assert (util.to_f64(outs[0])[~keep] == 0.0).all()


@pytest.mark.parametrize("M,N", [(1, 8), (1000, 8), (777, 24), (5, 64), (4001, 64), (333, 72), (129, 128), (77, 200), (1030, 256)])
@pytest.mark.parametrize("red", ["row_logsumexp", "row_softmax", "row_sum", "row_max", "row_mean"])
def test_elementwise_narrow_rows_share_a_warp(fc, orc, M, N, red):
    """Rows of at most 256 columns: a lane per 8-column chunk, 32 / cpr rows per warp (cpr = chunks per row rounded
    up to a power of two: 24 columns leave a lane of every four idle, 200 columns seven of 32), the row's pair
    merged inside its lane group.  Every reduction, with and without the main output, bf16 and fp16, ragged
    row counts, post ops, and -inf masks."""
    base = wl.affine_gelu_residual_lse(M, N)
    if red == "row_softmax":
        run_and_check(fc, orc, replace(base, reduce=red, store_main=False), 4)
        run_and_check(fc, orc, _as_f16(wl.scale_add_softmax(M, N)), 4)
        sm = wl.scale_add_softmax(M, N)
        ins = wl.make_inputs(sm, 6)
        keep = (np.arange(N)[None, :] + np.arange(M)[:, None]) % 5 != 0
        keep[:, 0] |= ~keep.any(axis=1)
        ins[1] = rng.store(np.where(keep, 0.0, -np.inf).astype(np.float32), "bf16")
        outs, _, _ = run_and_check(fc, orc, sm, ins=ins)
        assert (util.to_f64(outs[0])[~keep] == 0.0).all()
    else:
        run_and_check(fc, orc, replace(base, reduce=red, store_main=True), 4)
        run_and_check(fc, orc, replace(base, reduce=red, store_main=False, ops=(("bias_n", 2), ("relu",), ("scale", 0.5), ("clamp", -1.0, 1.0))), 4)
        run_and_check(fc, orc, _as_f16(replace(base, reduce=red, store_main=False, ops=())), 4)


@pytest.mark.parametrize("M,N", [(9, 50257), (17, 12289), (5, 10243), (3, 30001), (4, 20002)])
@pytest.mark.parametrize("dt", ["bf16", "f16"])
def test_elementwise_long_ragged_rows(fc, orc, M, N, dt):
    """A vocabulary of 50257: rows whose length is no multiple of 8 start anywhere in memory.  Chains without
    per-column vectors take the CTA-per-row kernel all the same: the aligned middle of every row in 16-byte chunks,
    up to 14 edge elements one by one.  Softmax (with a -inf mask too), logsumexp with the main output stored,
    sum / max / mean."""
    sm = wl.scale_add_softmax(M, N, dtype=dt)
    if dt == "bf16":
        run_and_check(fc, orc, sm, 3)
    ins = wl.make_inputs(sm, 5)
    keep = (np.arange(N)[None, :] * 7 + np.arange(M)[:, None]) % 640 < 3
    keep[:, [0, N - 1]] = True
    ins[1] = rng.store(np.where(keep, 0.0, -np.inf).astype(np.float32), dt)
    outs, _, _ = run_and_check(fc, orc, sm, ins=ins)
    assert (util.to_f64(outs[0])[~keep] == 0.0).all()
    base = replace(sm, ops=(("scale", 0.5), ("gelu_tanh",), ("add_tensor", 1)))
    run_and_check(fc, orc, replace(base, reduce="row_logsumexp", store_main=True), 3)
    for red in ("row_sum", "row_max", "row_mean"):
        run_and_check(fc, orc, replace(base, reduce=red, store_main=False, ops=(("relu",),)), 3)


def test_gelu_accuracy_dense_grid_fp32(fc, orc):
    """The kernels evaluate tanh-GELU with the hardware tanh approximation.  On a dense grid of
    inputs (fp32 in, fp32 out, so nothing but the activation's own error shows) the result must stay
    within 2e-5 of the fp64 value, five times inside the fp32 output tolerance at |ref| = 0."""
    n = 1 << 20
    x = np.linspace(-14.0, 14.0, n, dtype=np.float32).reshape(256, n // 256)
    ch = replace(wl.affine_gelu_residual_lse(256, n // 256), ops=(("gelu_tanh",),), reduce="none", in_dtype="f32", out_dtype="f32",
                 input_recipe=(("x", "f32", x.shape, "normal", 0.0, 1.0),))
    outs, ref, _ = run_and_check(fc, orc, ch, ins=[x])
    assert float(np.abs(util.to_f64(outs[0]) - ref["main"]).max()) <= 2e-5


@pytest.mark.parametrize("red", ["row_sum", "row_max", "row_mean"])
@pytest.mark.parametrize("M,N,dt", [(33, 4096, "bf16"), (7, 1000, "bf16"), (5, 333, "bf16"), (9, 515, "f32"), (64, 8192, "bf16")])
def test_elementwise_row_sum_max_mean(fc, orc, red, M, N, dt):
    base = wl.affine_gelu_residual_lse(M, N)
    rec = tuple((t, dt, s, d, a, b) for t, _, s, d, a, b in base.input_recipe)
    run_and_check(fc, orc, replace(base, reduce=red, in_dtype=dt, out_dtype=dt, input_recipe=rec), 4)
    run_and_check(fc, orc, replace(base, reduce=red, store_main=False, ops=(("relu",),), in_dtype=dt, out_dtype=dt, input_recipe=rec), 4)


def test_lse_shift_overflow_safety(fc, orc):
    ch = replace(wl.affine_gelu_residual_lse(4, 512), ops=(), in_dtype="f32", out_dtype="f32",
                 input_recipe=(("x", "f32", (4, 512), "normal", 0.0, 1.0),))
    x = wl.make_inputs(ch, 0)[0]
    x[1] += 1.0e4
    x[2] -= 1.0e4
    x[3, :] = -3.0
    x[3, 17] = 60.0
    run_and_check(fc, orc, ch, ins=[x])


def test_lse_row_dominated_by_one_gelu_value(fc, orc):
    """Adversarial for an approximate activation: one moderate GELU value dominates the row (every
    other residual is -30), so the logsumexp equals that value and inherits its full error."""
    ch = replace(wl.affine_gelu_residual_lse(64, 512), store_main=False)   # y itself is ~ -30: only the fp32 reduction is checked
    x, g, b, r = wl.make_inputs(ch, 9)
    rf = np.full((64, 512), -30.0, np.float32)
    cols = (np.arange(64) * 7) % 512
    rf[np.arange(64), cols] = 0.0
    xf = rng.bf16_bits_to_f32(x).copy()
    xf[np.arange(64), cols] = np.linspace(-3.0, 3.0, 64, dtype=np.float32)
    run_and_check(fc, orc, ch, ins=[rng.store(xf, "bf16"), g, b, rng.store(rf, "bf16")])


def _row_blocks(M, step):
    return [(r0, min(M, r0 + step)) for r0 in range(0, M, step)]


def test_c2_full_size_every_element(fc, orc):
    """The benchmark workload itself, in the launch configuration the benchmark times, every element of both
    outputs against the oracle (in blocks of rows, which are independent problems, to bound host memory)."""
    ch = wl.CONFIGS["C2"]()
    ins = wl.make_inputs(ch, 0)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    y, lse = outs[0].cpu(), outs[1].cpu()
    for r0, r1 in _row_blocks(ch.M, 2048):
        ref = orc.run_chain(replace(ch, M=r1 - r0), [ins[0][r0:r1], ins[1], ins[2], ins[3][r0:r1]])
        util.check(y[r0:r1], ref["main"], f"C2 y rows {r0}..{r1}")
        util.check(lse[r0:r1], ref["reduce"], f"C2 logsumexp rows {r0}..{r1}")


# ------------------------------------------------------------------ kernel (b): tcgen05 GEMM + epilogue
def _plain_gemm(M, N, K, out_dtype="f32"):
    return replace(wl.gemm_bias_gelu_scale_clamp(M, N, K), ops=(), out_dtype=out_dtype,
                   input_recipe=wl.gemm_bias_gelu_scale_clamp(M, N, K).input_recipe[:2])


@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (128, 256, 512), (256, 512, 128), (384, 768, 4096),
                                   (200, 264, 72), (1, 8, 8), (130, 40, 200), (128, 128, 64), (77, 100, 136)])
def test_gemm_tc_small_integers_bit_exact(fc, orc, M, N, K):
    """Integer operands (exact in bf16, partial sums < 2^24): any correct contraction gives the same
    bits, so the tensor-core path must equal the fp64 oracle exactly; exposes any layout permutation."""
    ch = wl.with_integer_inputs(_plain_gemm(M, N, K), -4, 4)
    ins = wl.make_inputs(ch, 5)
    ref = orc.run_chain(ch, ins)["main"]
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    got = util.to_f64(outs[0])
    assert np.array_equal(got, ref), f"{np.count_nonzero(got != ref)} of {got.size} elements differ"


def test_gemm_tc_one_hot_rows(fc, orc):
    M, N, K = 256, 512, 192
    ch = _plain_gemm(M, N, K)
    A = np.zeros((M, K), np.float32)
    A[np.arange(M), (np.arange(M) * 7) % K] = 1.0       # row m selects column (7m mod K) of B^T
    B = rng.integers_f32(0, "onehot/B", (N, K), -100, 100)
    ins = [rng.store(A, "bf16"), rng.store(B, "bf16")]
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    want = B[:, (np.arange(M) * 7) % K].T.astype(np.float64)
    assert np.array_equal(util.to_f64(outs[0]), want)


@pytest.mark.parametrize("variant", ["std", "var"])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_c3_chain_reduced(fc, orc, seed, variant):
    run_and_check(fc, orc, wl.gemm_bias_gelu_scale_clamp(512, 1024, 512, variant), seed)


@pytest.mark.parametrize("M,N,K", [(200, 264, 72), (129, 8, 8), (1000, 1000, 200)])
def test_c3_chain_ragged(fc, orc, M, N, K):
    run_and_check(fc, orc, wl.gemm_bias_gelu_scale_clamp(M, N, K, "var"), 4)
    run_and_check(fc, orc, replace(wl.gemm_bias_gelu_scale_clamp(M, N, K, "var"), out_dtype="f32"), 4)


@pytest.mark.parametrize("M,N,K", [(1000, 4000, 128), (1000, 3999, 72), (2048, 4096, 64), (1100, 3856, 200)])
def test_gemm_240_column_tiles(fc, orc, M, N, K):
    """Where rounds x tile width is smaller with 240-column tiles (two accumulators of 240 columns in tensor memory,
    epilogue halves of 128 and 112 columns) the GEMM kernels take them: a ragged last tile, rows off 16-byte
    boundaries, an exact multiple of 240 (3856 = 16 x 240 + 16: a last tile of one chunk), all three epilogues."""
    ch = wl.gemm_bias_gelu_scale_clamp(M, N, K, "var")
    run_and_check(fc, orc, ch, 21)
    assert fc.fc_last_plan() == "gemm_tc_mode0_bn240"
    run_and_check(fc, orc, replace(ch, out_dtype="f32"), 21)
    run_and_check(fc, orc, wl.gemm_bias_scale_lse(M, N, K, "var", True), 22)
    assert fc.fc_last_plan() == "gemm_tc_mode3_bn240"
    run_and_check(fc, orc, wl.linear_row_reduce(M, N, K, "row_max", ops=(("bias_n", 2), ("relu",)), store_main=False), 22)
    assert fc.fc_last_plan() == "gemm_tc_mode3_bn240"


@pytest.mark.parametrize("width", [128, 240, 256])
def test_one_shape_on_every_tile_width(fc, orc, width):
    """The testing switch FC_TESTING_TILE_WIDTH pins the column-tile width: the same ragged shapes through the plain
    store (bf16 and fp32 output), the row reductions, the single-pass softmax and the fp32 form on 128-, 240- and
    256-column tiles."""
    b = fc.binding
    b.fc_testing_set(b.FC_TESTING_TILE_WIDTH, width)
    try:
        M, N, K = 600, 1000, 264
        ch = wl.gemm_bias_gelu_scale_clamp(M, N, K, "var")
        run_and_check(fc, orc, ch, 31)
        assert fc.fc_last_plan().startswith(f"gemm_tc_mode0_bn{width}")
        run_and_check(fc, orc, replace(ch, out_dtype="f32"), 31)
        run_and_check(fc, orc, replace(wl.gemm_bias_gelu_scale_clamp(M, 999, K, "var"), out_dtype="f32"), 31)
        run_and_check(fc, orc, wl.gemm_bias_scale_lse(M, N, K, "var", True), 32)
        assert fc.fc_last_plan().startswith(f"gemm_tc_mode3_bn{width}")
        run_and_check(fc, orc, wl.linear_row_reduce(M, N, K, "row_max", ops=(("bias_n", 2), ("relu",)), store_main=False), 32)
        outs, _, _ = run_and_check(fc, orc, wl.gemm_softmax(M, N, K, "var"), 33)
        assert fc.fc_last_plan().startswith(f"gemm_tc_mode1_bn{width}") and "two_pass" not in fc.fc_last_plan()
        _check_softmax_rows(outs[0])
        run_and_check(fc, orc, wl.gemm_bias_relu_f32(1030, 1100, 512, "var"), 34)
        assert f"gemm_tc_mode7_bn{width}" in fc.fc_last_plan()
    finally:
        b.fc_testing_set(b.FC_TESTING_TILE_WIDTH, 0)


@pytest.mark.parametrize("M,N", [(520, 4000), (600, 3999), (777, 3856)])
def test_gemm_softmax_240_column_tiles(fc, orc, M, N):
    """The single-pass row softmax on 240-column tiles: 17 tiles per panel, the last one ragged."""
    ch = wl.gemm_softmax(M, N, 4096)
    run_and_check(fc, orc, ch, 23)
    assert fc.fc_last_plan() == "gemm_tc_mode1_bn240"
    run_and_check(fc, orc, replace(ch, out_dtype="f32"), 23)


@pytest.mark.parametrize("M,N,K,plan", [(100, 1000, 4096, "bn128_split"), (2048, 1024, 1024, "bn128"), (250, 2304, 768, "bn128"),
                                        (16, 8192, 4096, "bn128"), (16, 4096, 8192, "bn256_split"), (1024, 1024, 8192, "bn256_split")])
def test_gemm_few_tiles_either_tile_width(fc, orc, M, N, K, plan):
    """A GEMM of few tiles takes 128- or 256-column tiles, whole or cut along K, whichever a cost model makes
    faster: every combination against the oracle, bf16 and fp32 output."""
    ch = wl.gemm_bias_gelu_scale_clamp(M, N, K, "var")
    run_and_check(fc, orc, ch, 9)
    assert fc.fc_last_plan() == "gemm_tc_mode0_" + plan
    run_and_check(fc, orc, replace(ch, out_dtype="f32"), 9)


@pytest.mark.parametrize("M,N,K,plan", [(100, 1000, 4096, "bn128_split"), (300, 1100, 512, "bn128"), (1024, 4096, 1024, "bn240"),
                                        (64, 4096, 8192, "bn256_split")])
@pytest.mark.parametrize("store_main", [False, True])
def test_gemm_row_reduction_few_tiles_either_tile_width(fc, orc, M, N, K, plan, store_main):
    """The same choice for a row reduction behind the GEMM: per-tile partial results of 128- or 256-column tiles,
    whole or cut along K, merged per row."""
    run_and_check(fc, orc, wl.gemm_bias_scale_lse(M, N, K, "var", store_main), 10)
    assert fc.fc_last_plan() == "gemm_tc_mode3_" + plan
    run_and_check(fc, orc, wl.linear_row_reduce(M, N, K, "row_max", ops=(("bias_n", 2), ("relu",)), store_main=store_main), 10)


def test_gemm_tc_op_lists_fused_and_interpreted(fc, orc):
    """Op lists of the fused shape ([bias|affine] [relu|gelu] [scale] [clamp] [add tensor]) take the
    packed straight-line epilogue; any other order is interpreted op by op.  Both against the oracle."""
    base = wl.gemm_bias_gelu_scale_clamp(300, 520, 136, "var")
    rec = base.input_recipe + (("res", "bf16", (300, 520), "normal", 0.0, 1.0), ("gamma", "bf16", (520,), "normal", 1.0, 0.1))
    lists = [
        (("affine_n", 4, 2), ("relu",), ("scale", 1.5), ("clamp", 0.25, 2.0), ("add_tensor", 3)),       # fused
        (("bias_n", 2), ("gelu_tanh",), ("add_tensor", 3)),                                              # fused
        (("scale", -0.75),),                                                                             # fused (outputs stay O(1): the mean-abs bound is absolute)
        (("relu",), ("bias_n", 2), ("scale", 0.5), ("gelu_tanh",), ("add_tensor", 3), ("clamp", -1.0, 1.0)),  # interpreted
        (("clamp", -0.5, 0.5), ("affine_n", 4, 2), ("gelu_tanh",)),                                      # interpreted
    ]
    for ops in lists:
        for out_dtype in ("bf16", "f32"):
            run_and_check(fc, orc, replace(base, ops=ops, out_dtype=out_dtype, input_recipe=rec), 6, tag=f" ops={[o[0] for o in ops]}")


@pytest.mark.parametrize("N,res_dt", [(512, "bf16"), (520, "bf16"), (264, "f32"), (250, "bf16"), (250, "f32")])
def test_gemm_residual_rows_aligned_and_not(fc, orc, N, res_dt):
    """x + linear(x)-shaped chains: the residual row is read 16 columns at a time with 16-byte loads where its
    address allows (N a multiple of 8 for 16-bit storage, of 4 for fp32) and element by element otherwise
    (N = 250: odd rows start off a 16-byte boundary); the last, ragged chunk always goes element by element."""
    base = wl.gemm_bias_gelu_scale_clamp(300, N, 136, "var")
    rec = base.input_recipe + (("res", res_dt, (300, N), "normal", 0.0, 1.0),)
    for ops in [(("bias_n", 2), ("add_tensor", 3)), (("add_tensor", 3), ("relu",))]:
        run_and_check(fc, orc, replace(base, ops=ops, input_recipe=rec), 3)


@pytest.mark.parametrize("M,N,K", [(300, 250, 136), (129, 517, 72), (40, 33, 64), (513, 1001, 264)])
@pytest.mark.parametrize("out_dtype", ["bf16", "f32"])
def test_gemm_output_rows_off_16_byte_boundaries(fc, orc, M, N, K, out_dtype):
    """N that is no multiple of 8 (a vocabulary of 50257, say): output rows start anywhere, so the warp stores
    its block of rows together, 16 consecutive elements of two rows per instruction.  Plain store, softmax
    probabilities, and a stored main output beside a row reduction."""
    run_and_check(fc, orc, replace(wl.gemm_bias_gelu_scale_clamp(M, N, K, "var"), out_dtype=out_dtype), 2)
    run_and_check(fc, orc, replace(wl.gemm_softmax(M, N, K, "var"), out_dtype=out_dtype), 2)
    run_and_check(fc, orc, replace(wl.gemm_bias_scale_lse(M, N, K, store_main=True), out_dtype=out_dtype), 2)


@pytest.mark.parametrize("M,N,K,out_dtype", [(300, 20000, 72, "bf16"), (129, 16640, 136, "bf16"), (260, 16401, 64, "bf16"), (70, 16648, 64, "f32"),
                                             (130, 4400, 72, "bf16"), (257, 8190, 136, "f32"), (300, 8448, 4096, "bf16")])
def test_gemm_softmax_rows_wider_than_one_pass_allows(fc, orc, M, N, K, out_dtype):
    """More than 64 tiles per row panel: the SM pairs cannot hold a whole panel in tensor memory until its last
    tile arrives, so every tile stores its exponentials against its own maximum and a second kernel rescales
    the rows.  The same two-kernel form serves rows of more than 32 tiles, and of more than 16 behind a contraction
    shorter than 2048, where it is the faster one.  With ops and an additive -inf mask in front, aligned and
    unaligned rows, bf16 and fp32."""
    base = replace(wl.gemm_softmax(M, N, K, "var"), out_dtype=out_dtype)
    outs, _, _ = run_and_check(fc, orc, base, 5)
    assert fc.fc_last_plan().endswith("_two_pass softmax_rescale")
    np.testing.assert_allclose(util.to_f64(outs[0]).sum(1), 1.0, atol=3e-2 if out_dtype == "bf16" else 1e-4)
    rec = base.input_recipe + (("mask", "bf16", (M, N), "normal", 0.0, 1.0),)
    ch = replace(base, ops=(("scale", 0.5), ("add_tensor", 2)), input_recipe=rec)
    ins = wl.make_inputs(ch, 6)
    keep = np.arange(N)[None, :] <= (61 * np.arange(M)[:, None] + 3)
    ins[2] = rng.store(np.where(keep, 0.0, -np.inf).astype(np.float32), "bf16")
    outs, _, _ = run_and_check(fc, orc, ch, ins=ins)
    assert (util.to_f64(outs[0])[~keep] == 0.0).all()


def test_c3_full_size_every_element(fc, orc):
    """All 8192 x 8192 outputs of the benchmark's GEMM chain, in the launch configuration the benchmark times (32 pair
    panels x 32 column tiles over 74 CTA pairs, 14 rounds, L2 raster), against the oracle in blocks of 1024 rows."""
    ch = wl.CONFIGS["C3"]()
    ins = wl.make_inputs(ch, 0)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    got = outs[0].cpu()
    for r0, r1 in _row_blocks(ch.M, 1024):
        ref = orc.run_chain(replace(ch, M=r1 - r0), [ins[0][r0:r1], ins[1], ins[2]])
        util.check(got[r0:r1], ref["main"], f"C3 rows {r0}..{r1}")


# ------------------------------------------------------------------ kernel (c): GEMM + cross-tile row softmax
def _check_softmax_rows(t):
    s = t.float().sum(1)
    assert float((s - 1).abs().max()) <= 4e-3, "softmax rows must sum to 1 within bf16 rounding"


@pytest.mark.parametrize("variant", ["std", "var"])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (256, 1024, 256), (300, 1000, 136), (512, 4096, 128), (130, 264, 72),
                                   (300, 1000, 4096), (129, 4096, 4104), (600, 264, 4096)])   # the last three: single-pass form (K >= 4096)
def test_c4_softmax_reduced(fc, orc, M, N, K, variant):
    outs, _, _ = run_and_check(fc, orc, wl.gemm_softmax(M, N, K, variant), 1)
    _check_softmax_rows(outs[0])


def test_c4_softmax_dominant_logits(fc, orc):
    """A few logits per row far above the rest, in different column tiles: stresses the max merge."""
    ch = wl.gemm_softmax(256, 2048, 64, "var")
    A, B = wl.make_inputs(ch, 2)
    Af = rng.bf16_bits_to_f32(A).copy()
    Bf = rng.bf16_bits_to_f32(B).copy()
    Af[:, 0] = 8.0
    Bf[:, 0] = 0.0
    Bf[[5, 300, 900, 2047], 0] = [6.0, 6.25, 3.0, 6.25]     # +48..50 on columns in tiles 0, 1, 3, 7
    ins = [rng.store(Af, "bf16"), rng.store(Bf, "bf16")]
    outs, _, _ = run_and_check(fc, orc, ch, ins=ins)
    _check_softmax_rows(outs[0])


@pytest.mark.parametrize("M,N", [(300, 1000), (520, 4000)])
def test_gemm_softmax_single_pass_with_outliers(fc, orc, M, N):
    """Single-pass form (K >= 4096) with logits far above the rest: +20 / +35 / +50 in rising order inside one half
    row of a tile, in the second column half, in other tiles, in the last column; rows without any; then with the
    largest one in a half row's first 16 columns and falling ones behind it.  Stresses the maximum sweep, the
    exponentials against a half row's own maximum and the merge across halves and tiles."""
    ch = wl.gemm_softmax(M, N, 4096, "var")
    A, B = wl.make_inputs(ch, 2)
    Af = rng.bf16_bits_to_f32(A).copy()
    Bf = rng.bf16_bits_to_f32(B).copy()
    Af[:, 0] = 8.0
    Af[::3, 0] = 0.0                      # every third row: no outliers at all
    Bf[:, 0] = 0.0
    cols = {20: 2.5, 60: 4.375, 100: 6.25, 200: 6.0, 300: 6.25, 5 + 256: 3.0, N - 1: 6.25, N // 2 + 7: 5.0}
    for c, b in cols.items():
        Bf[c, 0] = b
    Af[1, 0] = 8.0
    ins = [rng.store(Af, "bf16"), rng.store(Bf, "bf16")]
    outs, _, _ = run_and_check(fc, orc, ch, ins=ins)
    assert fc.fc_last_plan().startswith("gemm_tc_mode1_bn") and "two_pass" not in fc.fc_last_plan()
    _check_softmax_rows(outs[0])
    # the largest outlier of the first half row in its first 16 columns, falling ones behind it
    Bf[:, 0] = 0.0
    for c, b in {3: 6.25, 40: 4.0, 90: 2.0, 130: 6.25, 140: 7.0}.items():
        Bf[c, 0] = b
    ins = [rng.store(Af, "bf16"), rng.store(Bf, "bf16")]
    outs, _, _ = run_and_check(fc, orc, ch, ins=ins)
    _check_softmax_rows(outs[0])


def test_gemm_softmax_single_pass_with_minus_infinity_mask(fc, orc):
    """The single-pass form behind scale + additive 0 / -inf mask: chunks, half rows and whole tiles of -inf in front
    of, between and behind the kept columns; masked probabilities are exactly 0."""
    M, N, K = 300, 1000, 4096
    base = wl.gemm_softmax(M, N, K, "var")
    rec = base.input_recipe + (("mask", "bf16", (M, N), "normal", 0.0, 1.0),)
    ch = replace(base, ops=(("scale", 0.5), ("add_tensor", 2)), store_main=False, input_recipe=rec)
    ins = wl.make_inputs(ch, 4)
    keep = np.arange(N)[None, :] <= (3 * np.arange(M)[:, None] + 2)
    keep[7] = False; keep[7, 600] = True
    keep[9] = np.arange(N) >= 900
    keep[11] = (np.arange(N) % 64) >= 48
    ins[2] = rng.store(np.where(keep, 0.0, -np.inf).astype(np.float32), "bf16")
    outs, ref, _ = run_and_check(fc, orc, ch, ins=ins)
    assert "two_pass" not in fc.fc_last_plan()
    got = util.to_f64(outs[0])
    assert (got[~keep] == 0.0).all()
    np.testing.assert_allclose(got.sum(1), 1.0, atol=2e-2)


@pytest.mark.parametrize("variant", ["std", "var"])
def test_c4_full_size_every_element(fc, orc, variant):
    """All 4096 x 4096 probabilities of the benchmark's GEMM + softmax chain (single-pass form, 16 tiles per row panel),
    under both readings of the input distribution."""
    ch = wl.gemm_softmax(variant=variant)
    assert (ch.M, ch.N, ch.K) == (4096, 4096, 4096)
    ins = wl.make_inputs(ch, 0)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    assert fc.fc_last_plan() == "gemm_tc_mode1_bn240"   # 18 tiles of 240 columns per panel: 288 tiles = 4 rounds on 72 pairs
    got = outs[0].cpu()
    for r0, r1 in _row_blocks(ch.M, 1024):
        ref = orc.run_chain(replace(ch, M=r1 - r0), [ins[0][r0:r1], ins[1]])
        util.check(got[r0:r1], ref["reduce"], f"C4 {variant} rows {r0}..{r1}")
    _check_softmax_rows(outs[0])


# ------------------------------------------------------------------ GEMM + row logsumexp (last tile of a panel merges)
@pytest.mark.parametrize("store_main", [False, True])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (300, 1000, 136), (256, 4096, 256), (130, 40, 72), (1024, 8200, 64)])
def test_gemm_row_logsumexp(fc, orc, M, N, K, store_main):
    run_and_check(fc, orc, wl.gemm_bias_scale_lse(M, N, K, "var", store_main), 3)


def test_gemm_row_logsumexp_dominant_and_repeat(fc, orc):
    """Dominant logits in different column tiles, and the same call twice (the scratch counters are
    re-zeroed per launch)."""
    ch = replace(wl.gemm_bias_scale_lse(256, 2048, 64, "var"), ops=())
    A, B, bias = wl.make_inputs(ch, 2)
    Af = rng.bf16_bits_to_f32(A).copy(); Bf = rng.bf16_bits_to_f32(B).copy()
    Af[:, 0] = 8.0; Bf[:, 0] = 0.0
    Bf[[5, 300, 900, 2047], 0] = [6.0, 6.25, 3.0, 6.25]
    ins = [rng.store(Af, "bf16"), rng.store(Bf, "bf16"), bias]
    for _ in range(2):
        run_and_check(fc, orc, ch, ins=ins)


# ------------------------------------------------------------------ kernel (d): implicit-GEMM conv + ReLU + avg-pool
def _delta_weights(C, r, s):
    w = np.zeros((C, 3, 3, C), np.float32)
    w[np.arange(C), r, s, np.arange(C)] = 1.0
    return rng.store(w, "bf16")


@pytest.mark.parametrize("r,s", [(1, 1), (0, 0), (2, 1), (0, 2)])
def test_conv_delta_kernels_pool_shifted_image(fc, orc, r, s):
    """A one-hot 3x3 kernel copies a shifted image, so the pooled output is the mean of ReLU(image)
    minus the row / column that falls off the edge: pins tap direction and zero padding."""
    ch = replace(wl.conv_bias_relu_avgpool(batch=3, H=10, W=12, Cin=64, Cout=64), ops=(("relu",),))
    x = wl.make_inputs(ch, 6)[0]
    run_and_check(fc, orc, ch, ins=[x, _delta_weights(64, r, s)])


@pytest.mark.parametrize("batch,H,W,Cin,Cout", [(1, 8, 16, 64, 64), (2, 14, 14, 64, 128), (3, 7, 9, 128, 256),
                                                (2, 56, 56, 64, 64), (5, 5, 5, 72, 40), (1, 1, 1, 8, 8)])
@pytest.mark.parametrize("seed", [0, 1])
def test_conv_chain_reduced(fc, orc, batch, H, W, Cin, Cout, seed):
    run_and_check(fc, orc, wl.conv_bias_relu_avgpool(batch=batch, H=H, W=W, Cin=Cin, Cout=Cout), seed)


@pytest.mark.parametrize("R,S,pad", [(1, 1, 0), (3, 3, 0), (5, 5, 2), (3, 5, 1), (5, 3, 2), (1, 3, 0), (7, 7, 3)])
def test_conv_filter_shapes(fc, orc, R, S, pad):
    """Filter sizes other than 3x3, non-square filters (pins which bounding-box corner belongs to
    which axis) and pad 0."""
    run_and_check(fc, orc, wl.conv_bias_relu_avgpool(batch=2, H=12, W=20, Cin=64, Cout=64, R=R, S=S, pad=pad), 5)


@pytest.mark.parametrize("R,S,pad,stride", [(1, 1, 0, 1), (3, 3, 1, 1), (5, 5, 0, 1), (5, 5, 2, 2), (3, 5, 1, 1), (7, 7, 3, 2), (4, 4, 1, 1)])
@pytest.mark.parametrize("pool", ["avg", "max"])
def test_conv_eight_channels_packs_filter_taps(fc, orc, R, S, pad, stride, pool):
    """Cin = 8 (an RGB image padded to 8 channels): a k-block holds eight filter taps, gathered as eight
    8-channel copies into an unswizzled operand tile; K = 8 R S ends inside a k-block for every shape here
    but 4 x 4, so the zero-filled tail chunks are exercised too.  Delta kernels pin the tap order."""
    make = wl.conv_bias_relu_avgpool if pool == "avg" else wl.conv_bias_relu_maxpool
    ch = make(batch=3, H=17, W=22, Cin=8, Cout=40, R=R, S=S, pad=pad, stride=stride)
    if pool == "max" and (ch.OH < 2 or ch.OW < 2):
        pytest.skip("no 2 x 2 window")
    run_without_workspace(fc, orc, ch, 9)
    if S == 1 or pad > 0:
        assert "gemm_tc_mode4" in fc.fc_last_plan()
    # with a workspace the padded shapes of more than one column run on a bordered copy of the image, a filter row per k-block
    run_and_check(fc, orc, ch, 9)
    if S > 1 and pad > 0:
        assert fc.fc_last_plan().startswith("pad_image ") and fc.fc_last_plan().endswith("_rowtaps")


@pytest.mark.parametrize("Cin,R,S,stride", [(8, 5, 5, 1), (8, 3, 3, 1), (16, 3, 3, 1), (8, 7, 7, 2), (32, 2, 2, 1), (16, 4, 4, 2), (24, 3, 2, 1), (8, 1, 8, 1),
                                             # rows of more than 64 elements, in 64-element pieces: 80, 96, 120 (two pieces), 72, 168 (three)
                                             (16, 5, 5, 1), (32, 3, 3, 1), (40, 3, 3, 1), (8, 3, 9, 1), (24, 2, 7, 2)])
@pytest.mark.parametrize("pool", ["avg", "max"])
def test_conv_few_channels_without_padding_takes_filter_rows(fc, orc, Cin, R, S, stride, pool):
    """Unpadded convolutions of few input channels: a k-block is one filter row (or a 64-element piece of one), fetched as one copy
    through a tensor map whose "pixels" are S * Cin channels wide and overlap (what the 64-element box asks for beyond
    them is out of range and arrives as zeros).  Ragged images, strides, both poolings; the last image's last rows sit
    at the end of the tensor."""
    make = wl.conv_bias_relu_avgpool if pool == "avg" else wl.conv_bias_relu_maxpool
    ch = make(batch=3, H=19, W=23, Cin=Cin, Cout=40, R=R, S=S, pad=0, stride=stride)
    run_and_check(fc, orc, ch, 11)
    assert fc.fc_last_plan().endswith("_rowtaps")
    # with padding the same shapes run on a bordered copy of the image (a layout pass into the workspace); without a
    # workspace they keep the tap-by-tap traversal
    if min(R, S) > 1:
        padded = make(batch=2, H=19, W=23, Cin=Cin, Cout=40, R=R, S=S, pad=1, stride=stride)
        run_and_check(fc, orc, padded, 11)
        # (where the pieces are more than half as many as the taps the border pass does not pay: tap by tap)
        pays = Cin == 8 or 2 * ((S * Cin + 63) // 64) <= S
        assert (fc.fc_last_plan().startswith("pad_image ") and fc.fc_last_plan().endswith("_rowtaps")) == pays
        run_without_workspace(fc, orc, padded, 11)
        assert "rowtaps" not in fc.fc_last_plan() and "pad_image" not in fc.fc_last_plan()


@pytest.mark.parametrize("Cin,R,S", [(8, 5, 5), (16, 5, 5), (32, 3, 3), (40, 3, 3), (24, 2, 7)])
def test_conv_filter_rows_delta_taps_bit_exact(fc, Cin, R, S):
    """One-hot filters pin which tap and channel every column of a filter-row k-block multiplies: output channel co
    copies input channel c shifted by (r, s), exactly (pooled ReLU of the shifted channel).  Rows of more than 64
    elements go in pieces: every piece of every row gets taps."""
    B, H, W = 2, 12, 14
    Cout = 3 * R * S + 5
    ch = replace(wl.conv_bias_relu_maxpool(batch=B, H=H, W=W, Cin=Cin, Cout=Cout, R=R, S=S, pad=0), ops=(("relu",),))
    ins = wl.make_inputs(ch, 4)
    x = rng.bf16_bits_to_f32(ins[0])
    w = np.zeros((Cout, R, S, Cin), dtype=np.float32)
    taps = [(co % (R * S) // S, co % (R * S) % S, (7 * co + co // (R * S)) % Cin) for co in range(Cout)]
    for co, (r, s, c) in enumerate(taps):
        w[co, r, s, c] = 1.0
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(ins[0]), fc.to_device(rng.store(w, "bf16"))], outs)
    fc.fc_get_async_status()
    assert fc.fc_last_plan().endswith("_rowtaps")
    OH, OW = H - R + 1, W - S + 1
    want = np.stack([np.maximum(x[:, r:r + OH, s:s + OW, c], 0) for r, s, c in taps], axis=-1)
    want = want[:, :OH // 2 * 2, :OW // 2 * 2].reshape(B, OH // 2, 2, OW // 2, 2, Cout).max(axis=(2, 4))
    assert np.array_equal(outs[0].cpu().numpy(), want)


def test_conv_eight_channels_delta_taps_bit_exact(fc):
    """One-hot filter (tap (r, s), channel c -> output channel): the max-pooled output is the pooled ReLU of a
    shifted image channel, exactly; every tap of a 5 x 5 filter in turn lands in a different chunk of the
    packed k-blocks."""
    B, H, W, R, S, pad = 2, 12, 14, 5, 5, 2
    ch = replace(wl.conv_bias_relu_maxpool(batch=B, H=H, W=W, Cin=8, Cout=32, R=R, S=S, pad=pad), ops=(("relu",),))
    ins = wl.make_inputs(ch, 4)
    x = rng.bf16_bits_to_f32(ins[0])
    w = np.zeros((32, R, S, 8), dtype=np.float32)
    taps = [(co % 25 // 5, co % 25 % 5, co % 8) for co in range(32)]
    for co, (r, s, c) in enumerate(taps):
        w[co, r, s, c] = 1.0
    xp = np.zeros((B, H + 2 * pad, W + 2 * pad, 8), dtype=np.float32)
    xp[:, pad:pad + H, pad:pad + W] = x
    want = np.stack([np.maximum(xp[:, r:r + H, s:s + W, c], 0) for r, s, c in taps], axis=-1)
    want = want.reshape(B, H // 2, 2, W // 2, 2, 32).max(axis=(2, 4))
    both = [ins[0], rng.store(w, "bf16")]
    outs = run_without_workspace(fc, None, ch, ins=both)      # eight taps per k-block
    assert "gemm_tc_mode4" in fc.fc_last_plan()
    assert np.array_equal(outs[0].cpu().numpy(), want)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in both], outs)    # bordered copy + a filter row per k-block
    fc.fc_get_async_status()
    assert fc.fc_last_plan().startswith("pad_image ")
    assert np.array_equal(outs[0].cpu().numpy(), want)


@pytest.mark.parametrize("H,W,R,S,pad,stride", [(12, 20, 3, 3, 1, 2), (13, 21, 3, 3, 1, 2), (16, 16, 1, 1, 0, 2), (15, 18, 5, 5, 2, 3), (14, 14, 3, 3, 0, 2)])
def test_conv_strided(fc, orc, H, W, R, S, pad, stride):
    run_and_check(fc, orc, wl.conv_bias_relu_avgpool(batch=3, H=H, W=W, Cin=64, Cout=64, R=R, S=S, pad=pad, stride=stride), 7)


def test_conv_all_ones_closed_form(fc, orc):
    ch = replace(wl.conv_bias_relu_avgpool(batch=2, H=56, W=56, Cin=256, Cout=256), ops=())
    x = rng.store(np.ones((2, 56, 56, 256), np.float32), "bf16")
    w = rng.store(np.ones((256, 3, 3, 256), np.float32), "bf16")
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(x), fc.to_device(w)], outs)
    fc.fc_get_async_status()
    np.testing.assert_allclose(util.to_f64(outs[0]), 2249.469387755102, rtol=1e-5)


def test_c5_full_size_every_element(fc, orc):
    """All 32 x 256 pooled outputs of the benchmark's convolution chain (392 pair tiles over 74 CTA pairs)."""
    ch = wl.CONFIGS["C5"]()
    ins = wl.make_inputs(ch, 0)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    ref = orc.run_chain(ch, ins)
    util.check(outs[0], ref["reduce"], "C5 (all images)")


# ------------------------------------------------------------------ host-buffer entry point
def test_run_host_matches_device_path(fc, orc):
    ch = wl.gemm_bias_gelu_scale_clamp(256, 512, 128, "var")
    ins = wl.make_inputs(ch, 3)
    host_in = [fc.to_device(a, "cpu").pin_memory() for a in ins]
    host_out = util.poison_(fc.binding.output_tensors(ch, "cpu", pinned=True))
    spec = fc.make_spec(ch)
    staging = torch.empty(fc.fc_staging_size(spec, host_in, host_out), dtype=torch.uint8, device="cuda")
    fc.run_chain_host(ch, host_in, host_out, staging)
    fc.fc_get_async_status()
    dev_out = fc.run_chain(ch, [t.cuda() for t in host_in])
    torch.cuda.synchronize()
    assert torch.equal(dev_out[0].cpu(), host_out[0])
    util.check(host_out[0], orc.run_chain(ch, ins)["main"], "fc_run_host")


def test_run_host_chunk_pipeline_matches_device_path(fc, orc):
    """Chains that move >= 32 MB go through fc_run_host's chunk pipeline (copies on two internal
    streams).  The results must equal those of the plain device path on the same inputs."""
    cases = [wl.affine_gelu_residual_lse(4100, 4096), wl.gemm_softmax(4096, 4096, 512, "var"),
             wl.gemm_bias_gelu_scale_clamp(4000, 4096, 512, "var"), wl.gemm_bias_scale_lse(4096, 4096, 512, "var", True),
             wl.conv_bias_relu_avgpool(batch=20), wl.conv_bias_relu_maxpool(batch=24, H=56, W=56, Cin=128, Cout=64, R=3, S=3, pad=1),
             wl.mlp(33000, (512, 256, 64)), wl.linear_row_reduce(20000, 1024, 1024),
             wl.scale_add_softmax(5000, 4096), wl.scale_add_softmax(300000, 64), wl.scale_add_softmax(700, 50257),
             wl.gemm_softmax(1100, 20000, 256, "var"), wl.conv_nchw(wl.conv_bias_relu_avgpool(batch=20)),
             wl.gemm_bias_relu_f32(3000, 3000, 1024, "var")]   # (fp32 on the tensor cores: whole tensors, no chunks)
    for ch in cases:
        ins = wl.make_inputs(ch, 1)
        host_in = [fc.to_device(a, "cpu").pin_memory() for a in ins]
        host_out = util.poison_(fc.binding.output_tensors(ch, "cpu", pinned=True))
        spec = fc.make_spec(ch)
        staging = torch.empty(fc.fc_staging_size(spec, host_in, host_out), dtype=torch.uint8, device="cuda")
        for _ in range(2):
            fc.run_chain_host(ch, host_in, host_out, staging)
        fc.fc_get_async_status()
        dev_out = fc.run_chain(ch, [t.cuda() for t in host_in])
        torch.cuda.synchronize()
        for a, b in zip(dev_out, host_out):
            if ch.reduce == "global_avgpool":      # pooled sums are combined with atomics: order varies
                assert torch.allclose(a.cpu(), b, rtol=1e-5, atol=1e-6)
            elif ch.producer == "gemm_nt" and ch.reduce == "row_softmax":
                # the same for the probabilities: a chunk of rows and the whole tensor may take tiles of different
                # widths (256 and 240 columns), i.e. other groupings of a row's partial sums: equal up to an ulp of
                # the 16-bit output here and there
                af, bf = a.cpu().float(), b.float()
                assert torch.allclose(af, bf, rtol=2 ** -7, atol=1e-9), ch.name
                assert (af == bf).float().mean() > 0.98, ch.name
            elif ch.producer == "gemm_nt" and ch.reduce == "row_logsumexp" and a.dim() == 1:
                # per-tile (max, sum) pairs are merged per row; the tile width depends on the row count of the
                # launch (a chunk of rows may take 128-column tiles where the whole tensor takes 256): same
                # terms, another grouping
                assert torch.allclose(a.cpu(), b, rtol=2e-6, atol=2e-6), ch.name
            else:
                assert torch.equal(a.cpu(), b), ch.name


# ------------------------------------------------------------------ fp16 storage (the paper's kernels store fp16)
def _as_f16(ch):
    rec = tuple((t, "f16" if d == "bf16" else d, sh, dist, a, b) for t, d, sh, dist, a, b in ch.input_recipe)
    return replace(ch, in_dtype="f16", out_dtype="f16" if ch.out_dtype == "bf16" else ch.out_dtype, input_recipe=rec)


def test_fp16_gemm_small_integers_bit_exact(fc, orc):
    for M, N, K in [(256, 512, 128), (200, 264, 72), (384, 768, 1024)]:
        ch = _as_f16(wl.with_integer_inputs(_plain_gemm(M, N, K), -4, 4))
        ins = wl.make_inputs(ch, 5)
        ref = orc.run_chain(ch, ins)["main"]
        outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
        fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
        fc.fc_get_async_status()
        assert np.array_equal(util.to_f64(outs[0]), ref)


@pytest.mark.parametrize("seed", [0, 1])
def test_fp16_chains(fc, orc, seed):
    run_and_check(fc, orc, _as_f16(wl.gemm_bias_gelu_scale_clamp(512, 1024, 512, "var")), seed)
    run_and_check(fc, orc, _as_f16(wl.gemm_bias_gelu_scale_clamp(200, 264, 72, "var")), seed)
    outs, _, _ = run_and_check(fc, orc, _as_f16(wl.gemm_softmax(300, 1000, 136, "var")), seed)
    assert float((outs[0].float().sum(1) - 1).abs().max()) <= 1e-3
    run_and_check(fc, orc, _as_f16(wl.gemm_bias_scale_lse(256, 2048, 256, "var", True)), seed)
    run_and_check(fc, orc, _as_f16(wl.conv_bias_relu_avgpool(batch=3, H=14, W=14, Cin=64, Cout=128)), seed)
    run_and_check(fc, orc, _as_f16(wl.affine_gelu_residual_lse(65, 4096)), seed)
    run_and_check(fc, orc, _as_f16(wl.affine_gelu_residual_lse(9, 1001)), seed)
    run_and_check(fc, orc, replace(_as_f16(wl.affine_gelu_residual_lse(33, 2048)), reduce="row_mean"), seed)


# ------------------------------------------------------------------ linear layer reduced over its output features
@pytest.mark.parametrize("red", ["row_sum", "row_max", "row_mean"])
@pytest.mark.parametrize("M,N,K,store_main", [(128, 256, 64, False), (300, 1000, 136, True), (256, 4096, 256, False), (130, 40, 72, True)])
def test_gemm_row_sum_max_mean_through_the_contraction(fc, orc, red, M, N, K, store_main):
    """A ReLU between the linear layer and the reduction keeps the GEMM: tensor-core kernel, per-tile
    partial results, last tile of a panel merges."""
    ch = wl.linear_row_reduce(M, N, K, red, ops=(("bias_n", 2), ("relu",), ("scale", 0.5)), variant="var", store_main=store_main)
    assert fc.binding.fc_describe_plan(fc.make_spec(ch))["kernel"] == "gemm_tc"
    run_and_check(fc, orc, ch, 8)


@pytest.mark.parametrize("red", ["row_sum", "row_mean"])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (300, 1000, 136), (77, 520, 4104), (1200, 264, 2048), (5000, 96, 512)])
@pytest.mark.parametrize("ops", [(), (("bias_n", 2),), (("bias_n", 2), ("scale", -0.75)), (("affine_n", 3, 4), ("bias_n", 2)),
                                 (("scale", 2.0), ("affine_n", 3, 4), ("scale", 0.5), ("bias_n", 2))])
def test_linear_row_sum_collapsed(fc, orc, red, M, N, K, ops):
    """Purely linear ops and no main output: the sum over the features is taken through the weights
    (out = A u + C); the oracle still does the full contraction."""
    ch = wl.linear_row_reduce(M, N, K, red, ops=ops, variant="var")
    assert fc.binding.fc_describe_plan(fc.make_spec(ch))["kernel"] == "collapse"
    run_and_check(fc, orc, ch, 9)


def test_linear_row_sum_collapsed_integer_inputs_exact(fc, orc):
    """Integer operands and no ops: every partial sum is an integer below 2^53, so the fp64 path gives
    the exact row sums; the fp32 output holds them exactly while they stay below 2^24."""
    ch = wl.with_integer_inputs(wl.linear_row_reduce(200, 512, 264, "row_sum", ops=()), -3, 3)
    ins = wl.make_inputs(ch, 3)
    outs, ref, _ = run_and_check(fc, orc, ch, ins=ins)
    assert np.abs(ref["reduce"]).max() < 2 ** 24
    np.testing.assert_array_equal(util.to_f64(outs[0]), ref["reduce"])


def test_linear_row_sum_fp16_collapsed_and_not(fc, orc):
    for ops in [(("bias_n", 2),), (("bias_n", 2), ("gelu_tanh",))]:
        ch = replace(wl.linear_row_reduce(256, 512, 256, "row_sum", ops=ops, variant="var"), in_dtype="f16", out_dtype="f16")
        ch = replace(ch, input_recipe=tuple((t, "f16", sh, d, a, b) for t, d0, sh, d, a, b in ch.input_recipe))
        run_and_check(fc, orc, ch, 10)


# ------------------------------------------------------------------ conv -> ReLU -> 2x2 max-pool
@pytest.mark.parametrize("batch,H,W,Cin,Cout,R,S,pad,stride", [
    (2, 8, 8, 64, 64, 3, 3, 1, 1), (3, 12, 20, 64, 128, 5, 5, 2, 1), (2, 9, 7, 64, 40, 3, 3, 1, 1), (1, 56, 56, 64, 256, 3, 3, 1, 1),
    (4, 5, 5, 72, 64, 1, 1, 0, 1), (2, 28, 28, 128, 64, 5, 5, 0, 1), (3, 17, 19, 64, 64, 3, 3, 1, 2), (5, 3, 2, 8, 8, 3, 3, 1, 1)])
def test_conv_relu_maxpool(fc, orc, batch, H, W, Cin, Cout, R, S, pad, stride):
    """Odd output sizes (dropped edge), windows that straddle warps and tiles, several images per tile."""
    ch = wl.conv_bias_relu_maxpool(batch=batch, H=H, W=W, Cin=Cin, Cout=Cout, R=R, S=S, pad=pad, stride=stride)
    for seed in (0, 1):
        run_and_check(fc, orc, ch, seed)


# (batch, H, W, Cin, Cout, R, S, pad): OH even and OW <= 64, so that tiles of whole row pairs exist; row pairs of 16, 20,
# 48, 56, 112 and 128 positions (128, 120, 96, 112, 112 and 128 positions per CTA), tiles across images, a last tile
# that ends inside its 128 positions, split last rounds (50 and 18 k-blocks), 64-, 128- and 256-column tiles
_WHOLE_PAIRS = [(5, 8, 8, 64, 64, 3, 3, 1), (7, 12, 10, 64, 128, 3, 3, 1), (2, 28, 28, 128, 64, 5, 5, 0), (3, 30, 30, 64, 136, 3, 3, 0),
                (2, 56, 56, 64, 256, 3, 3, 1), (3, 6, 64, 64, 72, 3, 3, 1), (9, 14, 14, 64, 128, 5, 5, 0), (4, 32, 32, 8, 64, 5, 5, 0),
                (3, 10, 9, 64, 48, 3, 3, 1)]


@pytest.mark.parametrize("shape", _WHOLE_PAIRS)
def test_conv_relu_maxpool_three_forms_agree(fc, orc, shape):
    """The 2 x 2 max-pool behind a convolution has three forms (every window through atomics; windows inside a tile
    finished on chip; tiles of whole row pairs, no atomics and no zeros in front).  A maximum is exact: all three
    give the same bits, and the oracle's values within the usual tolerance."""
    batch, H, W, Cin, Cout, R, S, pad = shape
    ch = wl.conv_bias_relu_maxpool(batch=batch, H=H, W=W, Cin=Cin, Cout=Cout, R=R, S=S, pad=pad)
    got = []
    try:
        for form in (1, 2, 3):
            fc.binding.fc_testing_set(fc.binding.FC_TESTING_POOL_FORM, form)
            outs, _, _ = run_and_check(fc, orc, ch, 21)
            assert ("zero_fill" in fc.fc_last_plan()) == (form != 3)
            got.append(outs[0].clone())
    finally:
        fc.binding.fc_testing_set(fc.binding.FC_TESTING_POOL_FORM, 0)
    assert torch.equal(got[0], got[1]) and torch.equal(got[0], got[2])


@pytest.mark.parametrize("dt", ["bf16", "f16"])
@pytest.mark.parametrize("shape", _WHOLE_PAIRS)
def test_conv_relu_maxpool_stored_in_16_bits(fc, orc, shape, dt):
    """out_dtype = bf16 / f16: the pooled output is stored in the next layer's operand type by the tile that holds the
    whole window.  Rounding is monotonic, so the result is the fp32 form's, rounded to nearest even, bit for bit."""
    batch, H, W, Cin, Cout, R, S, pad = shape
    base = wl.conv_bias_relu_maxpool(batch=batch, H=H, W=W, Cin=Cin, Cout=Cout, R=R, S=S, pad=pad)
    if dt == "f16":
        base = replace(base, in_dtype="f16", input_recipe=tuple((t, "f16", sh, d, a, b) for t, _, sh, d, a, b in base.input_recipe))
    ins = wl.make_inputs(base, 22)
    wide, _, _ = run_and_check(fc, orc, base, ins=ins)
    ch = replace(base, out_dtype=dt)
    outs, _, _ = run_and_check(fc, orc, ch, ins=ins)
    assert outs[0].dtype == (torch.bfloat16 if dt == "bf16" else torch.float16)
    assert "zero_fill" not in fc.fc_last_plan()
    assert torch.equal(outs[0], wide[0].to(outs[0].dtype))


def test_conv_relu_maxpool_16_bit_output_needs_whole_row_pairs(fc):
    for H, W in ((9, 8), (8, 130)):
        ch = replace(wl.conv_bias_relu_maxpool(batch=1, H=H, W=W, Cin=64, Cout=64, R=3, S=3, pad=1), out_dtype="bf16")
        ins = [fc.to_device(a) for a in wl.make_inputs(ch, 0)]
        with pytest.raises(fc.FcError, match="16-bit out_dtype"):
            fc.run_chain(ch, ins, fc.binding.output_tensors(ch, "cuda"))


def test_conv_relu_maxpool_delta_kernel_is_pooled_relu_of_image(fc, orc):
    """Centre-delta weights copy the image, so the output is the 2x2 max-pool of ReLU(image): compared
    with numpy on the stored bf16 values, exactly."""
    ch = replace(wl.conv_bias_relu_maxpool(batch=2, H=10, W=14, Cin=64, Cout=64, R=3, S=3, pad=1), ops=(("relu",),))
    x = wl.make_inputs(ch, 3)[0]
    outs, ref, _ = run_and_check(fc, orc, ch, ins=[x, _delta_weights(64, 1, 1)])
    img = np.maximum(rng.bf16_bits_to_f32(x).astype(np.float64), 0.0)
    want = img.reshape(2, 5, 2, 7, 2, 64).max(axis=(2, 4))
    np.testing.assert_array_equal(util.to_f64(outs[0]), want)


# ------------------------------------------------------------------ channel-first storage (CONV2D_NCHW)
@pytest.mark.parametrize("batch,H,W,Cin,Cout,R,S,pad,stride", [
    (2, 14, 14, 64, 128, 3, 3, 1, 1),
    (3, 9, 13, 72, 40, 3, 3, 1, 1),        # pixels and channels that are no multiple of the 64-wide transposition tile
    (1, 7, 7, 8, 8, 1, 1, 0, 1),           # one tap, fewest channels
    (5, 19, 11, 8, 72, 3, 5, 1, 2),        # 8 channels: eight filter taps per k-block, 15 taps = two blocks, the second one ragged
    (2, 23, 17, 136, 264, 5, 3, 2, 2),     # Cout over one 256-wide tile, strided, non-square filter
    (70, 8, 8, 64, 64, 3, 3, 1, 1),
])
@pytest.mark.parametrize("pool", ["avg", "max"])
def test_conv_channel_first(fc, orc, batch, H, W, Cin, Cout, R, S, pad, stride, pool):
    make = wl.conv_bias_relu_avgpool if pool == "avg" else wl.conv_bias_relu_maxpool
    ch = wl.conv_nchw(make(batch=batch, H=H, W=W, Cin=Cin, Cout=Cout, R=R, S=S, pad=pad, stride=stride))
    if pool == "max" and (ch.OH < 2 or ch.OW < 2):
        pytest.skip("no 2 x 2 window")
    run_and_check(fc, orc, ch, 21)
    # few channels with padding: the bordered copy of the image follows the channels-last rewrite
    short_rows = Cin < 64 and S > 1 and S * Cin <= 256 and (S * Cin + 63) // 64 < S
    assert ("pad_image" in fc.fc_last_plan()) == (short_rows and pad > 0 and (Cin == 8 or 2 * ((S * Cin + 63) // 64) <= S))
    assert fc.fc_last_plan().startswith("cfirst_to_clast cfirst_to_clast ")


def test_conv_channel_first_equals_channel_last_bitwise(fc):
    """The transposition moves bits: the pooled output of the channel-first chain is identical to the one of
    the channels-last chain on the permuted arrays (avg-pool accumulates with atomics, so compare the
    order-free max-pool)."""
    base = wl.conv_bias_relu_maxpool(batch=4, H=20, W=12, Cin=72, Cout=136, R=3, S=3, pad=1)
    ch = wl.conv_nchw(base)
    ins = wl.make_inputs(ch, 3)
    ins_cl = [np.ascontiguousarray(ins[0].transpose(0, 2, 3, 1)), np.ascontiguousarray(ins[1].transpose(0, 2, 3, 1))] + ins[2:]
    a = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    b = util.poison_(fc.binding.output_tensors(base, "cuda"))
    fc.run_chain(ch, [fc.to_device(x) for x in ins], a)
    fc.run_chain(base, [fc.to_device(x) for x in ins_cl], b)
    fc.fc_get_async_status()
    assert torch.equal(a[0], b[0])


@pytest.mark.parametrize("shape", [(4, 20, 12, 72, 136, 3, 3, 1), (3, 32, 32, 8, 64, 5, 5, 0), (70, 8, 8, 64, 64, 3, 3, 1)])
def test_conv_channel_first_pooled_in_16_bits(fc, orc, shape):
    """Channel-first operands with the max-pool stored in bf16: the layout pre-pass in front, tiles of whole row pairs
    behind it; the same bits as the channels-last chain on the permuted arrays, and the oracle's values."""
    batch, H, W, Cin, Cout, R, S, pad = shape
    base = replace(wl.conv_bias_relu_maxpool(batch=batch, H=H, W=W, Cin=Cin, Cout=Cout, R=R, S=S, pad=pad), out_dtype="bf16")
    ch = wl.conv_nchw(base)
    ins = wl.make_inputs(ch, 5)
    a, _, _ = run_and_check(fc, orc, ch, ins=ins)
    assert a[0].dtype == torch.bfloat16 and "zero_fill" not in fc.fc_last_plan()
    ins_cl = [np.ascontiguousarray(ins[0].transpose(0, 2, 3, 1)), np.ascontiguousarray(ins[1].transpose(0, 2, 3, 1))] + ins[2:]
    b = util.poison_(fc.binding.output_tensors(base, "cuda"))
    fc.run_chain(base, [fc.to_device(x) for x in ins_cl], b)
    fc.fc_get_async_status()
    assert torch.equal(a[0], b[0])
    # and through host buffers: the 16-bit pooled output comes back as it was stored
    host_in = [fc.to_device(x, "cpu").pin_memory() for x in ins_cl]
    outs = util.poison_(fc.binding.output_tensors(base, "cpu", pinned=True))
    staging = torch.empty(fc.fc_staging_size(fc.make_spec(base), host_in, outs), dtype=torch.uint8, device="cuda")
    fc.run_chain_host(base, host_in, outs, staging)
    fc.fc_get_async_status()
    assert torch.equal(outs[0], b[0].cpu())


def test_conv_channel_first_f16_and_host_path(fc, orc):
    ch = _as_f16(wl.conv_nchw(wl.conv_bias_relu_avgpool(batch=5, H=12, W=10, Cin=64, Cout=64)))
    run_and_check(fc, orc, ch, 2)
    ins = wl.make_inputs(ch, 2)
    ref = orc.run_chain(ch, ins)
    host_in = [fc.to_device(a, "cpu").pin_memory() for a in ins]
    outs = util.poison_(fc.binding.output_tensors(ch, "cpu", pinned=True))
    staging = torch.empty(fc.fc_staging_size(fc.make_spec(ch), host_in, outs), dtype=torch.uint8, device="cuda")
    fc.run_chain_host(ch, host_in, outs, staging)
    fc.fc_get_async_status()
    util.check(outs[0], ref["reduce"], "channel-first conv through host buffers")


def test_conv_channel_first_needs_workspace(fc):
    ch = wl.conv_nchw(wl.conv_bias_relu_avgpool(batch=2, H=8, W=8, Cin=64, Cout=64))
    ins = [fc.to_device(a) for a in wl.make_inputs(ch, 0)]
    outs = fc.binding.output_tensors(ch, "cuda")
    spec = fc.make_spec(ch)
    tiny = torch.empty(256, dtype=torch.uint8, device="cuda")
    fc.binding.fc_set_workspace(tiny)
    with pytest.raises(fc.FcError) as e:
        fc.binding.fc_run(spec, ins, outs)
    assert e.value.status == 6                        # FC_ERR_WORKSPACE


def test_maxpool_needs_relu_last(fc):
    import ctypes
    ch = replace(wl.conv_bias_relu_maxpool(), ops=(("bias_n", 2),))
    n = ctypes.c_size_t(0)
    assert fc.lib().fc_workspace_size(ctypes.byref(fc.make_spec(ch)), ctypes.byref(n)) == 3   # FC_ERR_UNSUPPORTED


def test_conv_relu_maxpool_fp16(fc, orc):
    ch = wl.conv_bias_relu_maxpool(batch=3, H=12, W=20, Cin=64, Cout=128, R=3, S=3, pad=1)
    ch = replace(ch, in_dtype="f16", input_recipe=tuple((t, "f16", sh, d, a, b) for t, _, sh, d, a, b in ch.input_recipe))
    run_and_check(fc, orc, ch, 4)


# ------------------------------------------------------------------ the further measured workloads at full size
@pytest.mark.parametrize("key", ["F1", "F2", "F3", "F4", "F5", "F6", "F7", "F8", "F9", "F11"])
def test_further_workloads_full_size_sampled(fc, orc, key):
    """Each workload the benchmark times beyond the five configurations, at its full size and in the launch
    configuration the benchmark uses; rows (images) are independent problems, so the oracle recomputes a sample
    of them: first and last, tile boundaries, and a stride through the rest."""
    ch = wl.ALL[key]()
    ins = wl.make_inputs(ch, 0)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    if ch.is_conv:
        pick = np.array([0, 17, ch.batch - 1])
        sub = replace(ch, batch=len(pick))
    else:
        pick = np.unique(np.concatenate([np.arange(0, ch.M, max(1, ch.M // 13) + 1), [0, 127, 128, 255, 256, ch.M - 1]]))
        sub = replace(ch, M=len(pick))
    per_row = {0} | {op[1] for op in ch.ops if op[0] == "add_tensor"}      # inputs with one row per problem
    sub_ins = [a[pick] if i in per_row else a for i, a in enumerate(ins)]
    ref = orc.run_chain(sub, sub_ins)
    sel = torch.from_numpy(pick).cuda()
    names = [r for r, _, _ in wl.output_shapes(ch)]
    for name, t in zip(names, outs):
        assert torch.isfinite(t.float()).all(), f"{key}: non-finite values in {name}"
        if any(op[0] == "linear" for op in ch.ops):
            util.check_chained(t[sel], ref[name], util.flip_allowance(orc, sub, sub_ins), f"{key} {name} (sampled rows)")
        else:
            util.check(t[sel], ref[name], f"{key} {name} (sampled)")
