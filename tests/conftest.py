import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle


@pytest.fixture(autouse=True)
def _guard_bands(request):
    """After every GPU test: no kernel wrote outside the tensors it was given (see tests/_util.py)."""
    if request.node.get_closest_marker("gpu") is None:
        yield
        return
    from _util import check_guards, guarded_empty
    from paper_2608_17641_b200 import binding
    plain = binding._alloc
    # outputs and workspaces that the binding allocates itself get bands too
    binding._alloc = lambda shape, dtype, device: guarded_empty(shape, dtype, label="allocated by the binding")
    try:
        yield
        check_guards(clear=True)
    finally:
        binding._alloc = plain
