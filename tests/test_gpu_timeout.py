"""The error path of the kernels' bounded waits, on the GPU, without a fault: a wait on a barrier that
nothing arrives on runs out after about a millisecond, the kernel returns, l4q_check reports
L4Q_ERR_TIMEOUT once, and the library keeps working in the same context."""
import pytest

from paper_2402_04902_b200 import binding as l4q
from paper_2402_04902_b200 import synth

import gpu_harness as gh

pytestmark = pytest.mark.gpu

L4Q_ERR_TIMEOUT = 5


def test_expired_wait_is_reported_and_the_context_stays_usable():
    gh.ensure_built()
    l4q.l4q_check()                                   # clean state
    l4q.l4q_selftest_timeout()
    with pytest.raises(l4q.L4QError) as e:
        l4q.l4q_check()
    assert e.value.status == L4Q_ERR_TIMEOUT
    l4q.l4q_check()                                   # reading the status cleared it
    # the same context still runs the layer, and reproducibly
    cfg = synth.LayerConfig("after_timeout", tokens=256, d_in=512, d_out=512, rank=16, alpha=32.0, bits=4,
                            group_size=128)
    arrays = synth.make_layer_inputs(cfg, seed=0)
    a = gh.run_layer(cfg, arrays, do_bwd=False)
    l4q.l4q_selftest_timeout()
    with pytest.raises(l4q.L4QError):
        l4q.l4q_check()
    b = gh.run_layer(cfg, arrays, do_bwd=False)
    assert (a["Y"] == b["Y"]).all()
