"""GPU parity of l4q_adamw_step (App. D) against the fp64 oracle over several steps."""
import numpy as np
import pytest
import torch

from oracle import l4q_oracle as orc
from paper_2402_04902_b200 import binding as l4q

import gpu_harness as gh

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n", [1, 1000, 16 * 4096 + 3])
def test_adamw_steps_match_the_oracle(n):
    gh.ensure_built()
    rng = np.random.default_rng(7)
    p0 = rng.normal(0, 0.05, n).astype(np.float32)
    p = gh.Guarded((n,), torch.float32); p.view.copy_(torch.from_numpy(p0))
    m = gh.Guarded((n,), torch.float32); m.view.zero_()
    v = gh.Guarded((n,), torch.float32); v.view.zero_()
    pr, mr, vr = p0.astype(np.float64), np.zeros(n), np.zeros(n)
    for step in range(1, 5):
        g = rng.normal(0, 1e-2, n).astype(np.float32)
        l4q.l4q_adamw_step(p.view, torch.from_numpy(g).cuda(), m.view, v.view, step, lr=2e-5 * 100, weight_decay=0.01)
        # the C ABI takes the hyper-parameters as float: the oracle gets the same (exactly widened) values
        f = lambda x: float(np.float32(x))
        pr, mr, vr = orc.adamw_step(pr, g.astype(np.float64), mr, vr, step, lr=f(2e-5 * 100), beta1=f(0.9),
                                    beta2=f(0.999), eps=f(1e-8), weight_decay=f(0.01))
    l4q.l4q_check()
    assert p.intact() and m.intact() and v.intact()
    assert np.allclose(p.view.double().cpu().numpy(), pr, rtol=1e-5, atol=1e-7)
    assert np.allclose(m.view.double().cpu().numpy(), mr, rtol=1e-5, atol=1e-9)
    assert np.allclose(v.view.double().cpu().numpy(), vr, rtol=1e-5, atol=1e-12)


def test_adamw_rejects_bad_arguments():
    gh.ensure_built()
    t = torch.zeros(8, dtype=torch.float32, device="cuda")
    with pytest.raises(l4q.L4QError) as e:
        l4q.l4q_adamw_step(t, t, t, t, 0, lr=1e-3)          # step counts from 1
    assert e.value.status == 1
