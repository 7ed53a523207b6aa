import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a) and the built CUDA library")


@pytest.fixture(scope="session")
def orc():
    import oracle
    oracle.build()
    return oracle


_BUILT = False


@pytest.fixture(autouse=True)
def _border_pass_at_any_size(request):
    """GPU tests run few-channel convolutions with padding on the bordered copy of the image whatever their size (the
    library takes that pass from some eight rounds of tiles on only: the test shapes are far smaller), so that the
    pass is exercised wherever a test has such a shape; tests of the size rule switch it back for themselves."""
    if request.node.get_closest_marker("gpu") is None:
        yield
        return
    import torch
    if not torch.cuda.is_available():
        yield
        return
    global _BUILT
    if not _BUILT:
        import __graft_entry__ as entry
        entry.build()
        _BUILT = True
    from paper_2602_14293_b200 import binding
    binding.fc_testing_set(binding.FC_TESTING_BORDER_PASS, 1)
    yield
    binding.fc_testing_set(binding.FC_TESTING_BORDER_PASS, 0)
