"""Tensors of more than 2^31 elements: every kernel's index arithmetic past the 32-bit range.

The oracle cannot walk such a tensor, so it computes sampled rows one by one (rows of these chains are
independent): the first and last rows, the rows on both sides of element 2^31 (and 2^32 where the tensor
reaches it) and a few in between.  Elementwise inputs repeat a seeded pattern of 4099 rows -- a prime, so a row
index that wrapped by a power of two lands on a different row of the pattern and fails the comparison.
Outputs are NaN-poisoned first and scanned afterwards: a row nobody wrote fails too.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

from fc_inputs import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu

PERIOD = 4099


@pytest.fixture(scope="module")
def fc():
    import __graft_entry__ as entry
    entry.build()
    import paper_2602_14293_b200 as fc
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    torch.cuda.set_device(0)
    return fc


def sample_rows(M, N):
    rows = {0, 1, PERIOD - 1, PERIOD, M // 3, M - 2, M - 1}
    for edge in (2 ** 31 // N, 2 ** 32 // N):
        for r in (edge - 1, edge, edge + 1):
            if 0 <= r < M:
                rows.add(r)
    return sorted(r for r in rows if 0 <= r < M)


def no_nan(t, what):
    flat = t.view(-1)
    for part in flat.split(1 << 28):
        assert not bool(torch.isnan(part).any()), f"{what}: elements left unwritten"


def check_rows(fc, orc, ch, outs, rows, small_ins, what):
    ref = orc.run_chain(replace(ch, M=len(rows)), small_ins)
    names = [r for r, _, _ in wl.output_shapes(ch)]
    idx = torch.tensor(rows, device=outs[0].device)
    for name, t in zip(names, outs):
        no_nan(t, f"{what}: {name}")
        util.check(t.index_select(0, idx), ref[name], f"{what}: {name} (rows {rows})")


def run_tiled_elementwise(fc, orc, ch, seed, what):
    """`ch`: an elementwise chain with more than 2^31 elements whose row-shaped inputs repeat a PERIOD-row pattern."""
    M, N = ch.M, ch.N
    assert M * N > 2 ** 31
    pat_recipe = tuple((t, d, (PERIOD, N) if len(s) == 2 else s, *rest) for t, d, s, *rest in ch.input_recipe)
    pattern = wl.make_inputs(replace(ch, M=PERIOD, input_recipe=pat_recipe), seed)
    reps = -(-M // PERIOD)
    ins = []
    for a in pattern:
        t = fc.to_device(a)
        ins.append(t.repeat(reps, 1)[:M] if t.dim() == 2 else t)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, ins, outs)
    fc.fc_get_async_status()
    rows = sample_rows(M, N)
    small = [a[[r % PERIOD for r in rows]] if a.ndim == 2 else a for a in pattern]
    check_rows(fc, orc, ch, outs, rows, small, what)
    del ins, outs
    torch.cuda.empty_cache()
    return fc.fc_last_plan()


def retype_f32(ch):
    rec = tuple((t, "f32", s, *rest) for t, _, s, *rest in ch.input_recipe)
    return replace(ch, in_dtype="f32", out_dtype="f32", input_recipe=rec)


def test_rows_kernel_past_2g(fc, orc):
    plan = run_tiled_elementwise(fc, orc, wl.affine_gelu_residual_lse(2 ** 19 + PERIOD + 5, 4096), 1, "warp per row")
    assert "ew_rows" in plan, plan


def test_rows_kernel_softmax_past_2g(fc, orc):
    plan = run_tiled_elementwise(fc, orc, wl.scale_add_softmax(2 ** 19 + 77, 4096), 2, "warp per row, softmax")
    assert "ew_rows" in plan, plan


def test_narrow_kernel_past_2g(fc, orc):
    plan = run_tiled_elementwise(fc, orc, wl.scale_add_softmax(2 ** 25 + PERIOD, 64), 3, "lane per chunk")
    assert "ew_narrow" in plan, plan


def test_longrow_kernel_past_2g(fc, orc):
    plan = run_tiled_elementwise(fc, orc, wl.affine_gelu_residual_lse(2 ** 17 + 1031, 16384), 4, "block per row")
    assert "ew_longrow" in plan, plan


def test_interpreter_flat_past_2g(fc, orc):
    ch = replace(retype_f32(wl.affine_gelu_residual_lse(2 ** 19 + 4111, 4096)), reduce="none")
    plan = run_tiled_elementwise(fc, orc, ch, 5, "interpreter, flat walk")
    assert "ew_interpreter" in plan, plan


def test_interpreter_rows_past_2g(fc, orc):
    ch = retype_f32(wl.affine_gelu_residual_lse(2 ** 19 + 4111, 4096))
    plan = run_tiled_elementwise(fc, orc, ch, 6, "interpreter, warp per row")
    assert "ew_interpreter" in plan, plan


def test_interpreter_block_rows_past_2g(fc, orc):
    ch = retype_f32(wl.scale_add_softmax(2 ** 17 + 1031, 16384))
    plan = run_tiled_elementwise(fc, orc, ch, 7, "interpreter, block per row, softmax")
    assert "ew_interpreter" in plan, plan


@pytest.mark.parametrize("kind", ["store", "logsumexp", "softmax"])
def test_gemm_output_past_2g(fc, orc, kind):
    M = N = 46400    # 2.15e9 output elements, 181.25 column tiles
    K = 64
    if kind == "store":
        ch = wl.gemm_bias_gelu_scale_clamp(M, N, K, "var")
    elif kind == "logsumexp":
        ch = wl.gemm_bias_scale_lse(M, N, K, "var", store_main=True)
    else:
        ch = wl.gemm_softmax(M, N, K, "var")
    assert M * N > 2 ** 31
    ins = wl.make_inputs(ch, 8)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    rows = sample_rows(M, N)
    small = [a[rows] if i == 0 else a for i, a in enumerate(ins)]
    check_rows(fc, orc, ch, outs, rows, small, f"gemm {kind}")
    del outs
    torch.cuda.empty_cache()
