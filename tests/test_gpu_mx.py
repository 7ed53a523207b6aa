"""GEMM chains on block-scaled 8-bit operands (MXFP8: E4M3 elements, one E8M0 scale per row and 32 elements along K)
against the CPU oracle, through the C ABI."""
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
    assert fc.fc_last_plan() == "scale_tiles scale_tiles gemm_tc_mode6_bn" + ("128" if ch.N <= 128 else "240")   # 256 x 240 tiles, 256 x 128 for narrow outputs
    util.check(outs[0], ref["main"], f"{ch.name} seed {seed}")
    return outs, ref


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (256, 512, 1024), (300, 520, 384), (1, 16, 128), (130, 40, 4096), (700, 136, 2176),
                                   (260, 240, 256), (257, 241, 256), (512, 960, 512), (100, 2000, 128)])
def test_mx_small_integers_and_power_of_two_scales_bit_exact(fc, orc, M, N, K):
    """Integer elements in [-4, 4] and block exponents in [-3, 3]: every product, block sum and scaled partial sum
    is exact in fp32, so the result must equal the fp64 oracle bit for bit.  A scale applied to the wrong row,
    column or block, or a permutation inside a k-block, would show."""
    ch = replace(wl.gemm_mxf8_bias_gelu_scale_clamp(M, N, K, out_dtype="f32", exp_lo=-3, exp_hi=3), ops=())
    r = np.random.default_rng(M + N + K)
    ins = wl.make_inputs(ch, 1)
    ins[0] = rng.store(r.integers(-4, 5, (M, K)).astype(np.float32), "f8e4m3")
    ins[1] = rng.store(r.integers(-4, 5, (N, K)).astype(np.float32), "f8e4m3")
    outs, ref = _run(fc, orc, ch, ins=ins)
    np.testing.assert_array_equal(util.to_f64(outs[0]), ref["main"])


def test_mx_every_scale_position_is_its_own(fc, orc):
    """Unit elements, and scales that differ for every (row, block) of A and every (column, block) of B: the output
    is 32 sum_j 2^(sa[m][j] + sb[n][j]), so a scale read from a neighbouring row, column or block changes it."""
    M, N, K = 256, 256, 512
    ch = replace(wl.gemm_mxf8_bias_gelu_scale_clamp(M, N, K, out_dtype="f32"), ops=())
    a = rng.store(np.ones((M, K), np.float32), "f8e4m3")
    b = rng.store(np.ones((N, K), np.float32), "f8e4m3")
    j = np.arange(K // 32)
    sa = ((np.arange(M)[:, None] * 7 + j[None, :] * 3) % 11 - 5).astype(np.float32)
    sb = ((np.arange(N)[:, None] * 5 + j[None, :]) % 9 - 4).astype(np.float32)
    outs, ref = _run(fc, orc, ch, ins=[a, b, rng.store(sa, "e8m0"), rng.store(sb, "e8m0")])
    np.testing.assert_array_equal(util.to_f64(outs[0]), ref["main"])
    want = 32.0 * (2.0 ** sa.astype(np.float64) @ (2.0 ** sb.astype(np.float64)).T)
    np.testing.assert_array_equal(ref["main"], want)


@pytest.mark.parametrize("M,N,K", [(256, 512, 512), (300, 520, 384), (1024, 1024, 4096)])
@pytest.mark.parametrize("out_dtype", ["bf16", "f32", "f16"])
def test_mx_chain(fc, orc, M, N, K, out_dtype):
    for seed in (3, 4):
        _run(fc, orc, wl.gemm_mxf8_bias_gelu_scale_clamp(M, N, K, out_dtype=out_dtype), seed)


def test_mx_extreme_scales(fc, orc):
    """Block exponents over a wide range (-40 .. 40 on both operands): products of scales from 2^-80 to 2^80 stay
    inside fp32, and blocks that are tiny next to others must still be added in."""
    ch = replace(wl.gemm_mxf8_bias_gelu_scale_clamp(200, 264, 640, out_dtype="f32", exp_lo=-40, exp_hi=40), ops=())
    ins = wl.make_inputs(ch, 6)
    ref = orc.run_chain(ch, ins)["main"]
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    got = util.to_f64(outs[0])
    # the outputs span many orders of magnitude: relative to each row's largest entry instead of 1 + |ref|
    scale = np.abs(ref).max(axis=1, keepdims=True)
    assert np.isfinite(got).all() and float((np.abs(got - ref) / scale).max()) <= 1e-5


def test_mx_rejections(fc):
    ch = wl.gemm_mxf8_bias_gelu_scale_clamp(256, 256, 96)        # K no multiple of 128
    ins = [fc.to_device(a) for a in wl.make_inputs(ch, 0)]
    with pytest.raises(fc.FcError) as err:
        fc.run_chain(ch, ins)
    assert err.value.status == 5
    ch = replace(wl.gemm_mxf8_bias_gelu_scale_clamp(256, 256, 128), reduce="row_softmax", store_main=False)
    with pytest.raises(fc.FcError) as err:
        fc.run_chain(ch, [fc.to_device(a) for a in wl.make_inputs(ch, 0)])
    assert err.value.status == 3
    ch = wl.gemm_mxf8_bias_gelu_scale_clamp(256, 256, 128)
    ins = [fc.to_device(a) for a in wl.make_inputs(ch, 0)]
    ins[2] = ins[2][:, :3].contiguous()                          # scale tensor of the wrong shape
    with pytest.raises(fc.FcError) as err:
        fc.run_chain(ch, ins)
    assert err.value.status == 4


def test_mx_host_path_and_graph_replay(fc, orc):
    """The same chain through fc_run_host (host tensors, staging buffer: all four producer inputs travel, also at a
    size that other chains would cut into row chunks) and, on the device, captured into a CUDA graph and replayed
    (three launches: two scale-tile kernels and the GEMM)."""
    for M, N, K in ((300, 264, 384), (6000, 2048, 2048)):
        ch = wl.gemm_mxf8_bias_gelu_scale_clamp(M, N, K)
        ins = wl.make_inputs(ch, 8)
        ref = orc.run_chain(ch, ins)["main"]
        host_in = [fc.to_device(a, "cpu").pin_memory() for a in ins]
        host_out = util.poison_(fc.binding.output_tensors(ch, "cpu", pinned=True))
        spec = fc.make_spec(ch)
        staging = torch.empty(fc.fc_staging_size(spec, host_in, host_out), dtype=torch.uint8, device="cuda")
        fc.run_chain_host(ch, host_in, host_out, staging)
        fc.fc_get_async_status()
        util.check(host_out[0], ref, f"mx fc_run_host {M}x{N}x{K}")
    dev = [t.cuda() for t in host_in]
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, dev, outs)                       # first call: one-time set-up outside the capture
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        fc.fc_run(spec, dev, outs, torch.cuda.current_stream())
    for _ in range(2):
        util.poison_(outs)
        graph.replay()
        torch.cuda.synchronize()
        util.check(outs[0], ref, "mx graph replay")
    fc.fc_get_async_status()
