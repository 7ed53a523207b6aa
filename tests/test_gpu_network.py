"""A network run as a sequence of fused chains (the paper's Level-3 example: conv -> ReLU -> max-pool twice, then
three linear layers), every stage on the GPU feeding the next without leaving the device.

Each stage is checked against the oracle ON THE INPUT THE GPU STAGE ACTUALLY SAW (the previous stage's GPU
output, copied back bit for bit), with that stage's usual tolerance: this pins shapes, layouts and conversions
of the composition without letting 16-bit rounding picks of one stage count against the next.  The final
logits are also compared with an oracle-only pass through the whole network, loosely (see the test)."""
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


def _to_numpy(t: torch.Tensor) -> np.ndarray:
    """Device tensor -> the stored form the oracle reads (float32, or uint16 bf16 bit patterns)."""
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def _out_name(ch):
    return wl.output_shapes(ch)[0][0]


@pytest.mark.parametrize("pooled", ["bf16", "f32"])
@pytest.mark.parametrize("batch", [64, 37])
def test_lenet_shaped_network_stage_by_stage(fc, orc, batch, pooled):
    stages = wl.lenet_shaped(batch, pooled=pooled)
    assert len(stages) == (3 if pooled == "bf16" else 5)
    prev_gpu = None          # GPU output of the previous stage
    prev_ref = None          # oracle-only pass: stored form of the previous stage's oracle output
    launches = fc.fc_launch_count()
    for k, ch in enumerate(stages):
        ins = wl.make_inputs(ch, 11 + k)
        dev_ins = [fc.to_device(a) for a in ins]
        if prev_gpu is not None:
            shape = ch.input_recipe[0][2]
            dev_ins[0] = prev_gpu.reshape(shape)                     # same bytes, no copy
            assert dev_ins[0].data_ptr() == prev_gpu.data_ptr()
            ins_seen = [_to_numpy(dev_ins[0])] + ins[1:]
            ins_ref = [prev_ref.reshape(shape)] + ins[1:]
        else:
            ins_seen = ins_ref = ins
        outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
        fc.run_chain(ch, dev_ins, outs)
        fc.fc_get_async_status()
        name = _out_name(ch)
        ref = orc.run_chain(ch, ins_seen)[name]
        if ch.name == "lenet_fc":
            util.check_chained(outs[0], ref, util.flip_allowance(orc, ch, ins_seen), f"stage {k} {ch.name}")
        else:
            util.check(outs[0], ref, f"stage {k} {ch.name}")
        if ch.name.startswith("cast"):
            # a conversion has one right answer: round to nearest even, bit for bit
            assert np.array_equal(_to_numpy(outs[0]), rng.f32_to_bf16_bits(ins_seen[0]))
        # oracle-only pass through the network, stored in each stage's output type
        full = orc.run_chain(ch, ins_ref)[name]
        out_dt = wl.output_shapes(ch)[0][1]
        prev_ref = rng.store(full.astype(np.float32), out_dt)
        prev_gpu = outs[0]
    assert fc.fc_launch_count() - launches >= len(stages)
    # End to end: the two passes differ only by rounding picks on the way; the logits stay close in norm and
    # nearly every row keeps its largest logit.
    got = util.to_f64(prev_gpu)
    want = full
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    assert rel < 2e-2, rel
    agree = (got.argmax(1) == want.argmax(1)).mean()
    assert agree >= 0.95, agree
