"""GPU parity of l4q_init_params (App. B) and l4q_quant_error (Table 4) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import l4q_oracle as orc
from paper_2402_04902_b200 import binding as l4q
from paper_2402_04902_b200 import synth

import gpu_harness as gh
import parity_utils as pu

pytestmark = pytest.mark.gpu

CASES = [
    synth.LayerConfig("init_bf16", tokens=8, d_in=1408, d_out=200, rank=16, alpha=32.0, bits=4, group_size=128),
    synth.LayerConfig("init_bf16_3bit", tokens=8, d_in=832, d_out=136, rank=8, alpha=16.0, bits=3, group_size=104,
                      signed_grid=True),
    synth.LayerConfig("init_f32", tokens=8, d_in=160, d_out=72, rank=5, alpha=10.0, bits=4, group_size=32,
                      io_dtype="f32"),
    synth.LayerConfig("init_wide_group", tokens=8, d_in=1024, d_out=64, rank=8, alpha=16.0, bits=4,
                      group_size=512),
    # the coalesced kernel at both ends of its range (1 and 32 lanes per group), with a ragged last warp,
    # and more pieces than one sweep of the grid covers
    synth.LayerConfig("init_group8", tokens=8, d_in=136, d_out=24, rank=8, alpha=16.0, bits=4, group_size=8,
                      signed_grid=True),
    synth.LayerConfig("init_group256", tokens=8, d_in=768, d_out=40, rank=8, alpha=16.0, bits=3, group_size=256),
    synth.LayerConfig("init_many_pieces", tokens=8, d_in=4096, d_out=2048, rank=8, alpha=16.0, bits=4,
                      group_size=64),
    # the TMA-fed kernel (bf16, groups of 32 / 64 / 128): a last column tile that is mostly beyond the weight and a
    # ragged last row tile; and enough tiles per CTA for the ring of stages to go round twice
    synth.LayerConfig("init_tma_ragged", tokens=8, d_in=1184, d_out=296, rank=8, alpha=16.0, bits=3, group_size=32,
                      signed_grid=True),
    synth.LayerConfig("init_tma_ring_wraps", tokens=8, d_in=8192, d_out=4096, rank=8, alpha=16.0, bits=4,
                      group_size=128),
]


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
@pytest.mark.parametrize("method", list(orc.INIT_METHODS))
def test_init_params_and_error_sums(cfg, method):
    gh.ensure_built()
    arrays = synth.make_layer_inputs(cfg, seed=21, need_acts=False)
    d = l4q.to_device(cfg, arrays)
    desc = l4q.make_desc(cfg)
    spec = pu.spec_of(cfg)
    G = cfg.d_in // cfg.group_size
    s = gh.Guarded((cfg.d_out, G), torch.float32)
    b = gh.Guarded((cfg.d_out, G), torch.float32)
    l4q.l4q_init_params(desc, d["W0"], method, s.view, b.view)
    l4q.l4q_check()
    assert s.intact() and b.intact()
    s_ref, b_ref = orc.init_params(spec, arrays["W0"].astype(np.float64), method)
    s_got, b_got = s.view.double().cpu().numpy(), b.view.double().cpu().numpy()
    assert np.allclose(s_got, s_ref, rtol=2e-6, atol=0)                      # fp32 reductions of <= 512 values
    assert np.allclose(b_got, b_ref, rtol=2e-6, atol=2e-6 * np.abs(s_ref).max())
    if method == "asymm" and not cfg.signed_grid:                            # b = group minimum, exactly
        assert np.array_equal(b_got, arrays["W0"].astype(np.float64).reshape(cfg.d_out, G, -1).min(axis=2))

    # error sums with the parameters the library just produced (so both sides quantize the same grid)
    err = torch.full((2,), float("nan"), dtype=torch.float64, device="cuda")
    s_dev, b_dev = s.view.contiguous(), b.view.contiguous()
    l4q.l4q_quant_error(desc, d["W0"], d["A"], d["B"], s_dev, b_dev, err)
    l4q.l4q_check()
    a = pu.widen(arrays)
    e_ref = orc.quant_error(spec, a["W0"], a["A"], a["B"], s_dev.double().cpu().numpy(), b_dev.double().cpu().numpy())
    e_got = err.cpu().numpy()
    print(cfg.name, method, e_got, e_ref)
    assert e_got[0] == pytest.approx(e_ref[0], rel=2e-5)
    # E_clip is a sum over few elements whose membership is a floating-point decision (see the STE gate):
    # one element more or less is possible, so compare within the largest single contribution
    tol = 2e-5 * e_ref[1] + 2.0 * np.abs(s_ref).max()
    assert abs(e_got[1] - e_ref[1]) <= tol


def test_asymm_and_l4q_init_do_not_clip_with_zero_B():
    # Table 4, "Initial": E_clip = 0.0
    gh.ensure_built()
    cfg = CASES[0]
    arrays = synth.make_layer_inputs(cfg, seed=22, need_acts=False, zero_B=True)
    d = l4q.to_device(cfg, arrays)
    desc = l4q.make_desc(cfg)
    G = cfg.d_in // cfg.group_size
    for method in ("asymm", "l4q"):
        s = torch.empty(cfg.d_out, G, dtype=torch.float32, device="cuda")
        b = torch.empty_like(s)
        err = torch.empty(2, dtype=torch.float64, device="cuda")
        l4q.l4q_init_params(desc, d["W0"], method, s, b)
        l4q.l4q_quant_error(desc, d["W0"], d["A"], d["B"], s, b, err)
        l4q.l4q_check()
        assert float(err[1]) == 0.0 and float(err[0]) > 0.0
