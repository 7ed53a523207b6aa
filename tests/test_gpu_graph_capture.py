"""fc_run inside CUDA graph capture: the call enqueues only (no allocation, no synchronisation), so a
captured chain replays correctly.  Launch-bound chains (C1's roofline time is 0.1 us) are the ones
that gain from replaying a graph instead of calling the library every step."""
from dataclasses import replace

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


@pytest.mark.parametrize("make", [
    lambda: wl.gemm_bias_relu_f32(256, 256, 256),
    lambda: wl.affine_gelu_residual_lse(64, 4096),
    lambda: wl.gemm_bias_gelu_scale_clamp(512, 512, 256, "var"),
    lambda: wl.gemm_softmax(256, 1024, 256, "var"),
    lambda: wl.gemm_bias_scale_lse(256, 1024, 256),
    lambda: wl.gemm_bias_gelu_scale_clamp(128, 256, 4096, "var"),          # split tiles
    lambda: wl.conv_bias_relu_avgpool(batch=2, H=14, W=14, Cin=64, Cout=128),
    lambda: wl.conv_bias_relu_maxpool(batch=3, H=15, W=14, Cin=64, Cout=128, R=3, S=3, pad=1),   # zero fill + atomics
    lambda: replace(wl.conv_bias_relu_maxpool(batch=9, H=14, W=14, Cin=8, Cout=64, R=5, S=5, pad=0), out_dtype="bf16"),   # one launch, pooled in bf16 (poisoned before every replay)
    lambda: wl.conv_bias_relu_avgpool(batch=5, H=17, W=15, Cin=8, Cout=64, R=5, S=5, pad=2),   # border pass into the workspace + zero fill + convolution
    lambda: wl.linear_row_reduce(96, 512, 256, variant="var"),             # three kernels
    lambda: wl.gemm_bias_relu_f32(1030, 1100, 512, "var"),                 # fp32 on the tensor cores: two split launches + the GEMM
    lambda: wl.gemm_softmax(600, 4000, 4096, "var"),                       # single-pass softmax on 240-column tiles
])
def test_captured_chain_replays(fc, orc, make):
    ch = make()
    ins = wl.make_inputs(ch, 21)
    ref = orc.run_chain(ch, ins)
    dev_ins = [fc.to_device(a) for a in ins]
    outs = fc.binding.output_tensors(ch, "cuda")
    spec = fc.make_spec(ch)
    fc.binding.ensure_workspace(spec)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        fc.fc_run(spec, dev_ins, outs)          # first call outside capture: one-time set-up of the library
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            fc.fc_run(spec, dev_ins, outs)
    names = [r for r, _, _ in wl.output_shapes(ch)]
    for _ in range(3):
        util.poison_(outs)
        graph.replay()
        torch.cuda.synchronize()
        for name, t in zip(names, outs):
            util.check(t, ref[name], f"graph replay {ch.name}: {name}")
    fc.fc_get_async_status()
