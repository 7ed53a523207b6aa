"""The allocation-free entry point against the ordinary one.

fc_run_softmax_static_scratch exists for callers that are handed tensors but cannot allocate a
workspace themselves (plug-ins without a memory pool, latency-critical loops where cudaMalloc is
off limits, processes whose device memory is reserved up front): it runs the GEMM + row-softmax kernel with
scratch from a fixed array inside the library.  Here it is called through the C ABI twice in a row,
on different inputs, and each result is compared with the fp64 CPU oracle of the chain and with what
fc_run (caller-provided workspace) writes for the same inputs, both within the bf16 tolerance of the
parity tests.  The second call also shows that what the first call left in the shared array does no harm.  This file sorts last so that
a run which stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from fc_inputs import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_fc_run_twice_in_a_row():
    import __graft_entry__ as entry
    entry.build()
    import paper_2602_14293_b200 as fc
    from paper_2602_14293_b200 import binding
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    torch.cuda.set_device(0)

    import oracle
    cases = [(wl.gemm_softmax(384, 1024, 256, "var"), 7), (wl.gemm_softmax(300, 2000, 136, "var"), 8)]
    for ch, seed in cases:
        spec = fc.make_spec(ch)
        host_ins = wl.make_inputs(ch, seed)
        ref = oracle.run_chain(ch, host_ins)["reduce"]       # the definition, in fp64 on the CPU
        ins = [fc.to_device(a) for a in host_ins]
        want = fc.run_chain(ch, ins)[0]                      # existing entry point, torch-owned workspace
        fc.fc_get_async_status()
        got = util.poison_(binding.output_tensors(ch, "cuda"))
        launches = fc.fc_launch_count()
        fc.fc_run_softmax_static_scratch(spec, ins, got)     # new entry point: nothing allocated
        fc.fc_get_async_status()
        assert fc.fc_launch_count() == launches + 1
        # the record of what was enqueued names this call's one kernel only (the single-pass softmax), not fc_run's
        assert fc.fc_last_plan() == "gemm_tc_mode1_bn256"
        util.check(got[0], ref, f"static scratch vs oracle ({ch.M}x{ch.N}x{ch.K})")
        util.check_bf16(util.to_f64(got[0]), util.to_f64(want), f"static scratch vs fc_run ({ch.M}x{ch.N}x{ch.K})")
        rows = got[0].float().sum(1)
        assert float((rows - 1).abs().max()) <= 4e-3

    # sizes beyond the built-in array are refused with a clear message, before anything is launched
    big = fc.make_spec(wl.gemm_softmax(8192, 8192, 64))
    assert fc.fc_workspace_size(big) > (1 << 20)
    a = torch.zeros(8192, 64, dtype=torch.bfloat16, device="cuda")
    out = torch.empty(8192, 8192, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(fc.FcError) as err:
        fc.fc_run_softmax_static_scratch(big, [a, a], [out])
    assert err.value.status == 6 and "built-in scratch holds" in str(err.value)
    # other chains are not served by it
    other = wl.gemm_bias_gelu_scale_clamp(256, 256, 64)
    with pytest.raises(fc.FcError) as err:
        fc.fc_run_softmax_static_scratch(fc.make_spec(other), [a[:256], a[:256], a[:256, 0].contiguous()],
                                         [out[:256, :256].contiguous()])
    assert err.value.status == 3
