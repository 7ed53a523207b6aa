"""GEMM chains with 8-bit E4M3 operands (fp32 accumulation on the tensor cores) against the CPU oracle."""
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


def _run(fc, orc, ch, seed=0, ins=None):
    if ins is None:
        ins = wl.make_inputs(ch, seed)
    ref = orc.run_chain(ch, ins)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    names = [r for r, _, _ in wl.output_shapes(ch)]
    for name, t in zip(names, outs):
        util.check(t, ref[name], f"{ch.name} seed {seed}: {name}")
    return outs, ref


@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (256, 512, 1024), (300, 520, 272), (1, 16, 16), (130, 40, 4096), (512, 128, 144)])
def test_f8_small_integers_bit_exact(fc, orc, M, N, K):
    """Integer operands in [-4, 4] are exact in E4M3 and every partial sum stays below 2^24: the result must
    equal the fp64 oracle bit for bit; any permutation inside the 128-wide k-blocks would show."""
    ch = replace(wl.gemm_f8_bias_gelu_scale_clamp(M, N, K, out_dtype="f32"), ops=())
    r = np.random.default_rng(M + N + K)
    ins = [rng.store(r.integers(-4, 5, (M, K)).astype(np.float32), "f8e4m3"),
           rng.store(r.integers(-4, 5, (N, K)).astype(np.float32), "f8e4m3"), wl.make_inputs(ch, 0)[2]]
    outs, ref = _run(fc, orc, ch, ins=ins)
    np.testing.assert_array_equal(util.to_f64(outs[0]), ref["main"])


@pytest.mark.parametrize("M,N,K", [(256, 512, 512), (300, 520, 272), (1024, 1024, 4096)])
@pytest.mark.parametrize("out_dtype", ["bf16", "f32"])
def test_f8_chain(fc, orc, M, N, K, out_dtype):
    _run(fc, orc, wl.gemm_f8_bias_gelu_scale_clamp(M, N, K, out_dtype=out_dtype), 3)


def test_f8_softmax_and_logsumexp(fc, orc):
    base = wl.gemm_f8_bias_gelu_scale_clamp(256, 1024, 512)
    soft = replace(base, name="gemm_f8_softmax", ops=(("scale", 1.0 / 512 ** 0.5),), reduce="row_softmax", store_main=False)
    _run(fc, orc, soft, 4)
    lse = replace(base, name="gemm_f8_lse", ops=(("scale", 1.0 / 512 ** 0.5), ("bias_n", 2)), reduce="row_logsumexp", store_main=False)
    _run(fc, orc, lse, 5)


def test_f8_split_tiles(fc, orc):
    ch = wl.gemm_f8_bias_gelu_scale_clamp(128, 256, 8192)
    spec = fc.make_spec(ch)
    fc.binding.ensure_workspace(spec)
    assert fc.binding.fc_describe_plan(spec)["split"] > 1
    _run(fc, orc, ch, 6)


def test_f8_rejections(fc):
    import ctypes
    n = ctypes.c_size_t(0)
    L = fc.lib()
    out_f8 = replace(wl.gemm_f8_bias_gelu_scale_clamp(64, 64, 64), out_dtype="f8e4m3")
    assert L.fc_workspace_size(ctypes.byref(fc.make_spec(out_f8)), ctypes.byref(n)) == 3     # FC_ERR_UNSUPPORTED
    ew = replace(wl.affine_gelu_residual_lse(64, 64), in_dtype="f8e4m3")
    assert L.fc_workspace_size(ctypes.byref(fc.make_spec(ew)), ctypes.byref(n)) == 3
