"""The bounds-checked build of the library (libfc_debug.so: the same sources with -DFC_DEBUG).

The memory checker that would normally vet the kernels' index arithmetic is not available on the machines this
repository is tested on, so the kernels can check themselves: every address that their own arithmetic produces for one
of their tensors is compared with that tensor's extent; a failed check skips the access and records FC_ERR_BOUNDS.
Here the ragged-shape parity cases run against that build in a child process (the library is chosen at import time)
and must pass with a clean status; a second child shows that a check which fails is reported and does no harm."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _debug_env():
    import __graft_entry__ as entry
    entry.build()
    from paper_2602_14293_b200 import build as fc_build
    lib = fc_build.build(debug=True)
    return dict(os.environ, FC_LIBRARY=lib)


def test_ragged_shapes_pass_the_address_checks():
    sel = ("ragged or shapes or reduced or strided or filter or maxpool or dominant or residual or odd or narrow or long or "
           "split or large_register or softmax_reduced or lse")
    out = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-k", sel, "tests/test_gpu_parity.py", "tests/test_gpu_split_tiles.py",
                          "tests/test_gpu_mx.py"], cwd=ROOT, env=_debug_env(), capture_output=True, text=True, timeout=1800)
    tail = out.stdout[-1500:] + out.stderr[-500:]
    assert out.returncode == 0, tail
    assert " passed" in out.stdout and "failed" not in out.stdout, tail


_TRIP = r"""
import sys
sys.path.insert(0, %r)
import torch
import paper_2602_14293_b200 as fc
from paper_2602_14293_b200 import binding
from fc_inputs import workloads as wl
from tests import util
assert binding.LIB_PATH.endswith("libfc_debug.so")
torch.cuda.set_device(0)
for ch in (wl.gemm_bias_gelu_scale_clamp(300, 520, 136, "var"), wl.affine_gelu_residual_lse(40, 4096)):
    ins = [fc.to_device(a) for a in wl.make_inputs(ch, 0)]
    outs = util.poison_(binding.output_tensors(ch, "cuda"))
    binding.fc_testing_set(binding.FC_TESTING_BOUNDS_TRIP, 1)      # the checks now believe the output to be one row shorter
    fc.run_chain(ch, ins, outs)
    try:
        fc.fc_get_async_status()
        raise SystemExit("no FC_ERR_BOUNDS for " + ch.name)
    except fc.FcError as e:
        assert e.status == 10 and "check site" in str(e), str(e)
    y = outs[0].float()
    assert torch.isnan(y[-1]).all(), "the last row was stored although its check failed"
    assert torch.isfinite(y[:-1]).all(), "rows inside the believed extent must be stored"
    binding.fc_testing_set(binding.FC_TESTING_BOUNDS_TRIP, 0)
    fc.run_chain(ch, ins, outs)
    fc.fc_get_async_status()                                       # clean again, and the device is usable
    assert torch.isfinite(outs[0].float()).all()
print("trip ok")
"""


def test_a_failed_check_is_reported_and_skips_the_access():
    out = subprocess.run([sys.executable, "-c", _TRIP % ROOT], cwd=ROOT, env=_debug_env(), capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "trip ok" in out.stdout, out.stdout[-1000:] + out.stderr[-1500:]
