"""Runs last (file name): after everything the GPU suite did in this process, no kernel has given up on a bounded wait
and - when the suite runs against the bounds-checking build (HE_DEBUG_LIB=1) - no index was out of range."""
import pytest

pytestmark = pytest.mark.gpu


def test_device_error_counter_is_still_zero():
    from paper_2412_16187_b200 import device_error_count
    assert device_error_count() == 0
