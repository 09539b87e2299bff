"""Collected after the other GPU tests: in a debug build of the library (LT_NVCC_FLAGS=-DLT_DEBUG_BOUNDS) the
compiled kernels have checked every address they formed in this process; none may have left its tensor.
In a release build the counter does not exist and the test is skipped."""
import pytest

pytestmark = pytest.mark.gpu


def test_compiled_kernels_stayed_inside_their_tensors():
    import paper_2102_13267_b200 as lt

    ctx = lt.LazyContext(device=0)
    n = ctx.debug_bounds_violations()
    ctx.close()
    if n is None:
        pytest.skip("release build: no bounds checks compiled in")
    assert n == 0
