"""Back-to-back linear layers kept on chip (LINEAR ops) against the CPU oracle, through the C ABI.

The oracle rounds the activation handed to the next layer onto the chain's 16-bit grid, as the kernel
does when it writes the next tensor-core operand; everything else is fp64.  Tolerances as for the
other 16-bit chains."""
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
    assert fc.binding.fc_describe_plan(fc.make_spec(ch))["kernel"] == "mlp_tc"
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    for _ in range(2):
        fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    assert tuple(outs[0].shape) == ref["main"].shape
    util.check_chained(outs[0], ref["main"], util.flip_allowance(orc, ch, ins), f"{ch.name} {ch.widths} seed {seed}")
    return outs, ref


@pytest.mark.parametrize("M,dims", [(128, (64, 64, 64)), (300, (64, 64, 64)), (1, (64, 16, 8)), (4096, (1024, 256, 256, 64)),
                                    (777, (400, 120, 88, 16)), (2048, (136, 256, 8)), (640, (72, 40, 200, 96, 24)), (20000, (256, 32, 16)), (1000, (400, 120, 88, 10)), (300, (64, 64, 3))])
def test_mlp_shapes(fc, orc, M, dims):
    _run(fc, orc, wl.mlp(M, dims, "std"), 1)


@pytest.mark.parametrize("act", ["relu", "gelu_tanh"])
@pytest.mark.parametrize("out_dtype", ["bf16", "f32"])
def test_mlp_activations_and_output_types(fc, orc, act, out_dtype):
    _run(fc, orc, wl.mlp(500, (192, 256, 128, 32), "std", act=act, out_dtype=out_dtype), 2)


def test_mlp_other_ops_between_layers(fc, orc):
    base = wl.mlp(384, (128, 64, 64, 32))
    # layer 1: affine + gelu + clamp; layer 2: bias + relu + scale; layer 3: nothing
    rec = list(base.input_recipe) + [("g", "bf16", (64,), "normal", 1.0, 0.1), ("be", "bf16", (64,), "normal", 0.0, 0.1)]
    ops = (("affine_n", 7, 8), ("gelu_tanh",), ("clamp", -0.5, 2.0), ("linear", 3), ("bias_n", 4), ("relu",), ("scale", 1.5), ("linear", 5))
    _run(fc, orc, replace(base, ops=ops, input_recipe=tuple(rec)), 3)


def test_mlp_fp16(fc, orc):
    ch = wl.mlp(300, (96, 128, 64), "std")
    ch = replace(ch, in_dtype="f16", out_dtype="f16", input_recipe=tuple((t, "f16", sh, d, a, b) for t, _, sh, d, a, b in ch.input_recipe))
    _run(fc, orc, ch, 4)


def test_mlp_small_integers_exact(fc, orc):
    """Integer inputs and weights small enough that every activation is an integer below 256 (exact in bf16)
    and every sum below 2^24: the result must equal the oracle bit for bit."""
    ch = replace(wl.mlp(260, (16, 16, 8, 8), out_dtype="f32"), ops=(("relu",), ("linear", 3), ("relu",), ("linear", 5)))
    ins = wl.make_inputs(ch, 5)
    r = np.random.default_rng(0)
    ins[0] = rng.store(r.integers(-2, 3, (260, 16)).astype(np.float32), "bf16")
    ins[1] = rng.store(r.integers(-2, 3, (16, 16)).astype(np.float32), "bf16")       # |h1| <= 64
    ins[3] = rng.store(r.integers(-1, 2, (8, 16)).astype(np.float32) * (r.random((8, 16)) < 0.25), "bf16")   # |h2| <= 64 * 16 / 4 on average; bounded below
    ins[5] = rng.store(r.integers(-2, 3, (8, 8)).astype(np.float32), "bf16")
    outs, ref = _run(fc, orc, ch, ins=ins)
    h1 = np.maximum(orc.widen(ins[0]) @ orc.widen(ins[1]).T, 0)
    h2 = np.maximum(h1 @ orc.widen(ins[3]).T, 0)
    assert h1.max() <= 256 and h2.max() <= 256, "the construction must keep the activations exact in bf16"
    np.testing.assert_array_equal(util.to_f64(outs[0]), ref["main"])


def test_mlp_identity_layers_copy_rounded_activations(fc, orc):
    """W2 = W3 = identity, no ops after layer 1: the output is layer 1's result rounded to bf16 (twice: a no-op)."""
    ch = replace(wl.mlp(256, (64, 64, 64, 64)), ops=(("linear", 3), ("linear", 5)))
    ins = wl.make_inputs(ch, 6)
    ins[3] = ins[5] = rng.store(np.eye(64, dtype=np.float32), "bf16")
    outs, ref = _run(fc, orc, ch, ins=ins)
    got, want = util.to_f64(outs[0]), ref["main"]
    # bf16 output of a value already on the bf16 grid: exact wherever both sides rounded layer 1 the same way
    assert np.mean(got == want) > 0.999


def test_mlp_rejections(fc):
    import ctypes
    n = ctypes.c_size_t(0)
    L = fc.lib()
    wide = wl.mlp(64, (64, 512, 64))          # hidden width 512 > 256
    assert L.fc_workspace_size(ctypes.byref(fc.make_spec(wide)), ctypes.byref(n)) == 3      # FC_ERR_UNSUPPORTED
    lse = replace(wl.mlp(64, (64, 64, 64)), reduce="row_logsumexp")
    assert L.fc_workspace_size(ctypes.byref(fc.make_spec(lse)), ctypes.byref(n)) == 3
