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


def test_adamw_multi_updates_the_four_tensors_of_a_layer_in_one_launch():
    """A, B, s, b of one layer (sizes that are no multiples of anything) in one launch, against the oracle tensor
    by tensor, over several steps; the launch counter moves by one per step."""
    gh.ensure_built()
    rng = np.random.default_rng(11)
    sizes = [16 * 4096, 11008 * 16 + 5, 11008 * 32 - 3, 7]
    dev, ref = [], []
    for n in sizes:
        p0 = rng.normal(0, 0.05, n).astype(np.float32)
        g = {k: gh.Guarded((n,), torch.float32) for k in ("p", "m", "v")}
        g["p"].view.copy_(torch.from_numpy(p0)); g["m"].view.zero_(); g["v"].view.zero_()
        dev.append(g)
        ref.append([p0.astype(np.float64), np.zeros(n), np.zeros(n)])
    f = lambda x: float(np.float32(x))
    for step in range(1, 4):
        grads = [rng.normal(0, 1e-2, n).astype(np.float32) for n in sizes]
        gd = [torch.from_numpy(g).cuda() for g in grads]
        n0 = l4q.l4q_launch_count()
        l4q.l4q_adamw_step_multi([(d["p"].view, gdk, d["m"].view, d["v"].view) for d, gdk in zip(dev, gd)], step,
                                 lr=2e-3, weight_decay=0.01)
        assert l4q.l4q_launch_count() - n0 == 1
        for r, g in zip(ref, grads):
            r[0], r[1], r[2] = orc.adamw_step(r[0], g.astype(np.float64), r[1], r[2], step, lr=f(2e-3), beta1=f(0.9),
                                              beta2=f(0.999), eps=f(1e-8), weight_decay=f(0.01))
    l4q.l4q_check()
    for d, r in zip(dev, ref):
        assert d["p"].intact() and d["m"].intact() and d["v"].intact()
        assert np.allclose(d["p"].view.double().cpu().numpy(), r[0], rtol=1e-5, atol=1e-7)
        assert np.allclose(d["m"].view.double().cpu().numpy(), r[1], rtol=1e-5, atol=1e-9)
        assert np.allclose(d["v"].view.double().cpu().numpy(), r[2], rtol=1e-5, atol=1e-12)
    with pytest.raises(l4q.L4QError) as e:
        t = torch.zeros(8, dtype=torch.float32, device="cuda")
        l4q.l4q_adamw_step_multi([(t, t, t, t)] * 9, 1, lr=1e-3)     # more than 8 tensors
    assert e.value.status == 1


def test_adamw_rejects_bad_arguments():
    gh.ensure_built()
    t = torch.zeros(8, dtype=torch.float32, device="cuda")
    with pytest.raises(l4q.L4QError) as e:
        l4q.l4q_adamw_step(t, t, t, t, 0, lr=1e-3)          # step counts from 1
    assert e.value.status == 1
