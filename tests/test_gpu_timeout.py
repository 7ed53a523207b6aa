"""The bounded device-side wait, exercised without any fault: a testing switch makes the row-softmax
kernel's cross-tile wait expect an arrival that never comes.  The wait must give up after its time
limit, the call must report FC_ERR_TIMEOUT through the status word instead of hanging, and the
next launch on the same device must work and be correct."""
import time

import numpy as np
import pytest
import torch

from fc_inputs import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


def test_panel_wait_expires_with_status_and_device_stays_usable(orc):
    import __graft_entry__ as entry
    entry.build()
    import paper_2602_14293_b200 as fc
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    torch.cuda.set_device(0)
    ch = wl.gemm_softmax(256, 512, 4096, "var")      # a long contraction: the single-pass form, whose tiles wait for their panel
    ins = wl.make_inputs(ch, 0)
    dev = [fc.to_device(a) for a in ins]
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.binding.fc_testing_set(fc.binding.FC_TESTING_PANEL_STALL, 1)
    try:
        t0 = time.perf_counter()
        fc.run_chain(ch, dev, outs)
        with pytest.raises(fc.FcError) as err:
            fc.fc_get_async_status()
        waited = time.perf_counter() - t0
    finally:
        fc.binding.fc_testing_set(fc.binding.FC_TESTING_PANEL_STALL, 0)
    assert err.value.status == 9                      # FC_ERR_TIMEOUT
    assert 1.5 <= waited <= 30.0, waited              # the limit is two seconds per wait
    assert torch.isnan(outs[0].float()).all()         # nothing was stored
    fc.fc_get_async_status()                          # the status word was cleared by the read
    ref = orc.run_chain(ch, ins)
    fc.run_chain(ch, dev, outs)
    fc.fc_get_async_status()
    util.check(outs[0], ref["reduce"], "softmax after an expired wait")


def test_split_merge_wait_expires_with_status_and_device_stays_usable(orc):
    """The merging slice of a split tile waits (bounded) for the slices that park their rows; with the
    testing switch it expects one arrival too many."""
    import __graft_entry__ as entry
    entry.build()
    import paper_2602_14293_b200 as fc
    torch.cuda.set_device(0)
    ch = wl.gemm_bias_gelu_scale_clamp(128, 256, 4096, "var")
    ins = wl.make_inputs(ch, 0)
    dev = [fc.to_device(a) for a in ins]
    spec = fc.make_spec(ch)
    fc.binding.ensure_workspace(spec)
    assert fc.binding.fc_describe_plan(spec)["split"] > 1
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.binding.fc_testing_set(fc.binding.FC_TESTING_SPLIT_STALL, 1)
    try:
        t0 = time.perf_counter()
        fc.run_chain(ch, dev, outs)
        with pytest.raises(fc.FcError) as err:
            fc.fc_get_async_status()
        waited = time.perf_counter() - t0
    finally:
        fc.binding.fc_testing_set(fc.binding.FC_TESTING_SPLIT_STALL, 0)
    assert err.value.status == 9                      # FC_ERR_TIMEOUT
    assert 1.5 <= waited <= 30.0, waited
    assert torch.isnan(outs[0].float()).all()         # the only tile was split: nothing was stored
    fc.fc_get_async_status()
    ref = orc.run_chain(ch, ins)
    for _ in range(2):                                # counters left behind by the expired launch are cleared
        util.poison_(outs)
        fc.run_chain(ch, dev, outs)
        fc.fc_get_async_status()
        util.check(outs[0], ref["main"], "split GEMM after an expired wait")
