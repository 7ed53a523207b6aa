"""Split tiles (K cut into slices when the output tiles do not fill the SM pairs) against the oracle.

Every case runs twice through the C ABI: with the workspace that allows splitting (the plan must then
report split > 1) and with only the workspace the chain requires (split == 1).  Both results are
checked against the CPU oracle with the usual tolerances; integer-valued inputs must agree bit for
bit whatever the summation order.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

from fc_inputs import workloads as wl
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


def _register(fc, spec, split):
    """Register a workspace that allows (split=True) or forbids (False) splitting; returns it."""
    b = fc.binding
    need = b.fc_workspace_size_split(spec) if split else b.fc_workspace_size(spec)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda") if need else None
    b.fc_set_workspace(ws)
    b._workspace.clear()   # the convenience cache no longer describes what is registered
    return ws


def _run_both(fc, orc, ch, seed=0, ins=None, expect_split=True):
    if ins is None:
        ins = wl.make_inputs(ch, seed)
    ref = orc.run_chain(ch, ins)
    dev_ins = [fc.to_device(a) for a in ins]
    spec = fc.make_spec(ch)
    names = [r for r, _, _ in wl.output_shapes(ch)]
    results = {}
    for split in (True, False):
        ws = _register(fc, spec, split)
        plan = fc.binding.fc_describe_plan(spec)
        assert plan["kernel"] == "gemm_tc"
        if split and expect_split:
            assert plan["split"] > 1 and plan["split_tiles"] > 0, plan
        if not split:
            assert plan["split"] == 1, plan
        outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
        for _ in range(2):   # twice: the counters must come back at zero without a memset
            fc.fc_run(spec, dev_ins, outs)
        fc.fc_get_async_status()
        for name, t in zip(names, outs):
            util.check(t, ref[name], f"{ch.name} split={split} seed {seed}: {name}")
        results[split] = [t.clone() for t in outs]
        del ws
    fc.binding.fc_set_workspace(None)
    return results, ref


@pytest.mark.parametrize("M,N,K", [(192, 1000, 4096), (128, 256, 4096), (256, 128, 4096), (520, 520, 4104), (1024, 1024, 8192)])
def test_small_m_gemm_epilogue(fc, orc, M, N, K):
    _run_both(fc, orc, wl.gemm_bias_gelu_scale_clamp(M, N, K, "var"), 11)


def test_tail_round_is_split(fc, orc):
    """80 tiles on 74 pairs: one full round, then 6 tiles cut into slices."""
    ch = wl.gemm_bias_gelu_scale_clamp(2560, 2048, 4096, "var")
    spec = fc.make_spec(ch)
    _register(fc, spec, True)
    plan = fc.binding.fc_describe_plan(spec)
    if plan["pairs"] != 74:
        pytest.skip(f"shape chosen for 74 pairs, this device runs {plan['pairs']}")
    assert plan["tiles"] == 80 and plan["split_tiles"] == 6 and plan["split"] > 1, plan
    _run_both(fc, orc, ch, 12)


@pytest.mark.parametrize("M,N,K", [(256, 512, 4096), (300, 1000, 4104)])
def test_split_integer_inputs_bit_exact(fc, orc, M, N, K):
    base = wl.gemm_bias_gelu_scale_clamp(M, N, K)
    ch = wl.with_integer_inputs(replace(base, name=f"gemm_plain_{M}x{N}x{K}", ops=(), out_dtype="f32", input_recipe=base.input_recipe[:2]), -4, 4)
    ins = wl.make_inputs(ch, 4)
    res, ref = _run_both(fc, orc, ch, ins=ins)
    for split in (True, False):
        np.testing.assert_array_equal(util.to_f64(res[split][0]), ref["main"])


@pytest.mark.parametrize("store_main", [False, True])
def test_split_row_logsumexp(fc, orc, store_main):
    _run_both(fc, orc, wl.gemm_bias_scale_lse(256, 2048, 4096, "var", store_main), 13)


def test_split_row_softmax_single_round(fc, orc):
    _run_both(fc, orc, wl.gemm_softmax(256, 1024, 4096, "var"), 14)


def test_softmax_of_several_rounds_is_not_split(fc, orc):
    ch = wl.CONFIGS["C4"]()
    spec = fc.make_spec(ch)
    _register(fc, spec, True)
    plan = fc.binding.fc_describe_plan(spec)
    assert plan["split"] == 1, plan
    fc.binding.fc_set_workspace(None)


@pytest.mark.parametrize("kind", ["store", "lse"])
def test_split_last_round_of_240_column_tiles(fc, orc, kind):
    """84 tiles of 256 x 240 on 74 pairs: one full round and ten tiles cut along K (the second warp group of a
    240-column tile has seven chunks: parked and merged slices must leave the eighth, the other buffer's, alone)."""
    M, N, K = 1536, 3360, 4096
    ch = wl.gemm_bias_gelu_scale_clamp(M, N, K, "var") if kind == "store" else wl.gemm_bias_scale_lse(M, N, K, "var", True)
    spec = fc.make_spec(ch)
    _register(fc, spec, True)
    plan = fc.binding.fc_describe_plan(spec)
    assert plan["bn"] == 240 and plan["split"] > 1 and 0 < plan["split_tiles"] < plan["tiles"], plan
    _run_both(fc, orc, ch, 17)


def test_split_fp16(fc, orc):
    ch = wl.gemm_bias_gelu_scale_clamp(192, 520, 4096, "var")
    ch = replace(ch, in_dtype="f16", out_dtype="f16", input_recipe=tuple((t, "f16", sh, d, a, b) for t, _, sh, d, a, b in ch.input_recipe))
    _run_both(fc, orc, ch, 16)


def test_split_conv_5x5(fc, orc):
    _run_both(fc, orc, wl.conv_bias_relu_avgpool(batch=1, H=16, W=16, Cin=128, Cout=64, R=5, S=5, pad=2), 15)


def test_alternating_layouts_and_repeats(fc, orc):
    """Two chains whose counters sit at different places of one workspace, called in turn."""
    a = wl.gemm_bias_scale_lse(256, 2048, 4096, "var", False)
    b = wl.gemm_bias_gelu_scale_clamp(192, 1000, 4096, "var")
    sa, sb = fc.make_spec(a), fc.make_spec(b)
    need = max(fc.binding.fc_workspace_size_split(sa), fc.binding.fc_workspace_size_split(sb))
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    ws.fill_(0xFF)   # whatever was there: the library clears what it needs
    fc.binding.fc_set_workspace(ws)
    fc.binding._workspace.clear()
    ia, ib = wl.make_inputs(a, 1), wl.make_inputs(b, 2)
    ra, rb = orc.run_chain(a, ia), orc.run_chain(b, ib)
    da, db = [fc.to_device(t) for t in ia], [fc.to_device(t) for t in ib]
    for _ in range(3):
        oa = util.poison_(fc.binding.output_tensors(a, "cuda"))
        ob = util.poison_(fc.binding.output_tensors(b, "cuda"))
        fc.fc_run(sa, da, oa)
        fc.fc_run(sb, db, ob)
        fc.fc_run(sb, db, ob)
        fc.fc_get_async_status()
        util.check(oa[0], ra["reduce"], "lse between other layouts")
        util.check(ob[0], rb["main"], "gemm between other layouts")
    fc.binding.fc_set_workspace(None)
