"""The failure path on a real device, without faulting it: a bounded device-side wait that runs out
sets the error word, convbn_check reports CONVBN_ETIMEOUT once, and the library keeps working."""
import pytest

import parity
from paper_2305_11624_b200 import convbn as C
from paper_2305_11624_b200 import inputs as I

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_once_and_the_context_stays_usable():
    C.convbn_check()                                   # start from a clean error word
    C.convbn_selftest_wait_timeout()
    with pytest.raises(C.ConvBNError) as e:
        C.convbn_check()
    assert e.value.status == C.ETIMEOUT
    C.convbn_check()                                   # the word was cleared by the failing check
    # a normal call afterwards runs and is correct
    spec = I.LayerSpec("after_timeout", 2, 64, 12, 16, 64, 3, 3, pad=1)
    t = parity.make_inputs(spec, 3)
    got = parity.run_tune_gpu(spec, t)                 # ends with convbn_check(): must be OK
    parity.compare(got, parity.oracle_tune(spec, t), parity.TOL["bf16"], parity.TUNE_OUTPUTS, spec.name, dtype="bf16")
