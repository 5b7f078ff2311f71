"""The device-side error path: a bounded wait inside a kernel that runs out must come back to the host as
DDTREE_ERR_DEVICE_TIMEOUT through ddtree_device_status(), once, with the context still usable.  The wait is
made to run out by construction (a barrier nothing arrives at, a bound of a few thousand polls): nothing
traps, faults or hangs."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_once_and_the_context_stays_usable():
    import paper_2604_12989_b200 as dd
    from tests import test_gpu_attention as ta
    dd.device_status()                      # clean before
    dd.selftest_wait_timeout()
    with pytest.raises(dd.DDTreeError) as e:
        dd.device_status()
    assert e.value.status == 5
    assert "wait" in str(e.value)
    dd.device_status()                      # reading the word cleared it
    # the context is still usable: a real attention call afterwards runs and matches the oracle
    w, att, trees = ta.bf16_case(1, 40, 8, 2, (300,))
    out, lse = ta.gpu_attention(w, att, trees)
    ta.compare(w, att, trees, out, lse)
    dd.device_status()
