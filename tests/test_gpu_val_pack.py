"""GPU parity: fp32 validation path (fwd, bwd) and the pack kernel against the fp64 oracle."""
import numpy as np
import pytest

from oracle import l4q_oracle as orc
from paper_2402_04902_b200 import synth
from paper_2402_04902_b200.synth import CONFIG1

import gpu_harness as gh
import parity_utils as pu

pytestmark = pytest.mark.gpu


def _check_fwd_bwd(cfg, arrays, out, grad_scale=1.0):
    spec = pu.spec_of(cfg, grad_scale)
    a = pu.widen(arrays)
    bf = cfg.io_dtype == "bf16"
    Y = orc.forward(spec, a["X"], a["W0"], a["A"], a["B"], a["s"], a["b"], bf16_reference=bf)
    g = orc.backward(spec, a["X"], a["dY"], a["W0"], a["A"], a["B"], a["s"], a["b"], bf16_reference=bf)
    assert pu.max_rel_err(out["Y"], Y) <= pu.TOL_OUT[cfg.io_dtype]
    assert pu.max_rel_err(out["dX"], g["dX"]) <= pu.TOL_OUT[cfg.io_dtype]
    for k in ("dA", "dB", "ds", "db"):
        assert pu.rel_l2(out[k], g[k]) <= pu.TOL_GRAD[cfg.io_dtype], k


def _check_pack(cfg, arrays, out):
    spec = pu.spec_of(cfg)
    a = pu.widen(arrays)
    w, wt, _ = orc.fake_quant_weight(spec, a["W0"], a["A"], a["B"], a["s"], a["b"])
    got_u = orc.unpack_int(spec, out["codes"], cfg.d_in)
    res = pu.check_codes(got_u, spec, w)
    assert res["out_of_band"] == 0, res
    assert res["mismatches"] <= res["allowed"], res
    _, s16, b16 = orc.pack_int(spec, a["W0"], a["A"], a["B"], a["s"], a["b"])
    assert np.array_equal(out["s16"].view(np.uint16), s16.view(np.uint16))
    assert np.array_equal(out["b16"].view(np.uint16), b16.view(np.uint16))


def test_config1_fp32_forward_backward():
    arrays = synth.make_layer_inputs(CONFIG1, seed=0)
    out = gh.run_layer(CONFIG1, arrays)
    _check_fwd_bwd(CONFIG1, arrays, out)


def test_config1_zero_B_equals_plain_quantization_of_W0():
    arrays = synth.make_layer_inputs(CONFIG1, seed=0, zero_B=True)
    out = gh.run_layer(CONFIG1, arrays, do_pack=True)
    _check_fwd_bwd(CONFIG1, arrays, out)
    _check_pack(CONFIG1, arrays, out)
    # B = 0: merge == W0, min/max init never clips -> db == 0 exactly up to in-band elements
    a = pu.widen(arrays)
    spec = pu.spec_of(CONFIG1)
    g = orc.backward(spec, a["X"], a["dY"], a["W0"], a["A"], a["B"], a["s"], a["b"])
    assert pu.rel_l2(out["db"], g["db"]) <= 1e-4 or np.abs(out["db"] - g["db"]).max() < 1e-3


@pytest.mark.parametrize("signed", [False, True])
@pytest.mark.parametrize("bits", [3, 4])
def test_fp32_ragged_shapes(signed, bits):
    # spans several 64-wide tiles with ragged tails in every dimension
    cfg = synth.LayerConfig("ragged_f32", tokens=75, d_in=200, d_out=136, rank=5, alpha=10.0, bits=bits,
                            group_size=40, io_dtype="f32", outliers=True, signed_grid=signed)
    if (cfg.d_in * bits) % 32:
        cfg = cfg.with_(d_in=160, group_size=32)
    arrays = synth.make_layer_inputs(cfg, seed=3)
    out = gh.run_layer(cfg, arrays, do_pack=True, grad_scale=0.5)
    _check_fwd_bwd(cfg, arrays, out, grad_scale=0.5)
    _check_pack(cfg, arrays, out)


@pytest.mark.parametrize("bits,rank,group", [(4, 16, 128), (3, 64, 64), (4, 8, 32), (3, 16, 32)])
@pytest.mark.parametrize("signed", [False, True])
def test_pack_bf16_weights(bits, rank, group, signed):
    # bf16 W0 with outliers; d_in = 1312 = 5 x 256 + 32 exercises a ragged column tile, d_out = 200 ragged rows
    cfg = synth.LayerConfig("pack_bf16", tokens=8, d_in=1312 if group == 32 else 1408, d_out=200, rank=rank,
                            alpha=32.0, bits=bits, group_size=group, io_dtype="bf16", signed_grid=signed)
    arrays = synth.make_layer_inputs(cfg, seed=5, need_acts=False)
    out = gh.run_layer(cfg, arrays, do_fwd=False, do_bwd=False, do_pack=True)
    _check_pack(cfg, arrays, out)


def test_skipping_outputs_and_error_codes():
    import torch
    from paper_2402_04902_b200 import binding as l4q
    gh.ensure_built()
    arrays = synth.make_layer_inputs(CONFIG1, seed=1)
    dev = l4q.to_device(CONFIG1, arrays)
    desc = l4q.make_desc(CONFIG1)
    outs = l4q.alloc_outputs(CONFIG1)
    ws = l4q.alloc_workspace(desc, l4q.L4Q_OP_BWD)
    # dX only
    l4q.l4q_linear_bwd(desc, dev["X"], dev["dY"], dev["W0"], dev["A"], dev["B"], dev["s"], dev["b"],
                       outs["dX"], None, None, None, None, ws)
    # parameter gradients only
    l4q.l4q_linear_bwd(desc, dev["X"], dev["dY"], dev["W0"], dev["A"], dev["B"], dev["s"], dev["b"],
                       None, outs["dA"], outs["dB"], outs["ds"], outs["db"], ws)
    l4q.l4q_check()
    a = pu.widen(arrays)
    g = orc.backward(pu.spec_of(CONFIG1), a["X"], a["dY"], a["W0"], a["A"], a["B"], a["s"], a["b"])
    assert pu.max_rel_err(outs["dX"].double().cpu().numpy(), g["dX"]) <= 1e-4
    assert pu.rel_l2(outs["dA"].double().cpu().numpy(), g["dA"]) <= 1e-4
    # three of four parameter gradients -> invalid argument; short workspace -> workspace error
    with pytest.raises(l4q.L4QError) as e:
        l4q.l4q_linear_bwd(desc, dev["X"], dev["dY"], dev["W0"], dev["A"], dev["B"], dev["s"], dev["b"],
                           None, outs["dA"], outs["dB"], outs["ds"], None, ws)
    assert e.value.status == 1
    with pytest.raises(l4q.L4QError) as e:
        l4q.l4q_linear_fwd(desc, dev["X"], dev["W0"], dev["A"], dev["B"], dev["s"], dev["b"], outs["Y"],
                           torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3
