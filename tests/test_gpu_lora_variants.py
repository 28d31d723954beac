"""GPU parity of the LoRA (Eq. 1-2) and QAT-LoRA (Sec. 3.1) layers against the fp64 oracle,
element by element: exact tiles, ragged tails in every dimension, every rank class, more tiles
than SMs, and the argument checks.  B is drawn large enough that the LoRA path carries about a
third of Y and dX (with the tiny B of a freshly initialised adapter an error in that path would
hide inside the tolerance)."""
import numpy as np
import pytest
import torch

from oracle import l4q_oracle as orc
from paper_2402_04902_b200 import binding as l4q
from paper_2402_04902_b200 import synth

import gpu_harness as gh
import parity_utils as pu

pytestmark = pytest.mark.gpu


def _inputs(cfg, seed):
    arrays = synth.make_layer_inputs(cfg, seed=seed)
    rng = np.random.default_rng(seed + 1000)
    arrays["B"] = rng.normal(0.0, 0.05, arrays["B"].shape).astype(np.float32)
    return arrays


def run_variant(cfg, arrays, kind, grad_scale=1.0, want_quant_grads=True):
    gh.ensure_built()
    M = arrays["X"].shape[0]
    desc = l4q.make_desc(cfg, grad_scale=grad_scale, tokens=M)
    dev = l4q.to_device(cfg, arrays)
    G = cfg.d_in // cfg.group_size
    qat = kind == l4q.L4Q_LORA_QAT
    s, b = (dev["s"], dev["b"]) if qat else (None, None)
    guards = {"Y": gh.Guarded((M, cfg.d_out), torch.bfloat16), "dX": gh.Guarded((M, cfg.d_in), torch.bfloat16),
              "dA": gh.Guarded((cfg.rank, cfg.d_in), torch.float32),
              "dB": gh.Guarded((cfg.d_out, cfg.rank), torch.float32)}
    if qat and want_quant_grads:
        guards["ds"] = gh.Guarded((cfg.d_out, G), torch.float32)
        guards["db"] = gh.Guarded((cfg.d_out, G), torch.float32)
    ws = l4q.alloc_lora_workspace(desc, kind, l4q.L4Q_OP_FWD)
    l4q.l4q_lora_linear_fwd(desc, kind, dev["X"], dev["W0"], dev["A"], dev["B"], s, b, guards["Y"].view, ws)
    ws = l4q.alloc_lora_workspace(desc, kind, l4q.L4Q_OP_BWD)
    l4q.l4q_lora_linear_bwd(desc, kind, dev["X"], dev["dY"], dev["W0"], dev["A"], dev["B"], s, b,
                            guards["dX"].view, guards["dA"].view, guards["dB"].view,
                            guards["ds"].view if "ds" in guards else None,
                            guards["db"].view if "db" in guards else None, ws)
    out = {}
    if qat:   # the codes of Q(W0): the export of the same quantizer with a zero LoRA factor
        pk = l4q.alloc_pack_outputs(cfg)
        l4q.l4q_pack_int(desc, dev["W0"], dev["A"], torch.zeros_like(dev["B"]), dev["s"], dev["b"], pk["codes"],
                         pk["s16"], pk["b16"])
        out["codes"] = pk["codes"].cpu().numpy().view(np.uint32)
    l4q.l4q_check()
    for k, g in guards.items():
        assert g.intact(), f"out-of-bounds write around {k}"
        out[k] = g.view.to(torch.float64).cpu().numpy()
    return out


def check_variant(cfg, arrays, kind, grad_scale=1.0):
    out = run_variant(cfg, arrays, kind, grad_scale)
    spec = pu.spec_of(cfg, grad_scale)
    a = pu.widen(arrays)
    if kind == l4q.L4Q_LORA_PLAIN:
        Y = orc.lora_forward(spec, a["X"], a["W0"], a["A"], a["B"], bf16_reference=True)
        g = orc.lora_backward(spec, a["X"], a["dY"], a["W0"], a["A"], a["B"], bf16_reference=True)
    else:
        qn, _ = orc.grid_bounds(spec)
        w = orc.prequant(spec, a["W0"], a["s"], a["b"])
        got_u = orc.unpack_int(spec, out["codes"], cfg.d_in)
        res = pu.check_codes(got_u, spec, w)
        # W0 alone on a grid initialised from its own min/max puts many weights exactly on a tie k + 1/2
        # (bf16 values, fp32 scale); both neighbours are correct there, so only off-tie mismatches count
        assert res["out_of_band"] == 0, res
        codes = got_u + qn
        Y = orc.qat_lora_forward(spec, a["X"], a["W0"], a["A"], a["B"], a["s"], a["b"], bf16_reference=True,
                                 codes=codes)
        g = orc.qat_lora_backward(spec, a["X"], a["dY"], a["W0"], a["A"], a["B"], a["s"], a["b"],
                                  bf16_reference=True, codes=codes)
    # the LoRA path must matter in this test: compare against the base product alone
    base = a["X"] @ a["W0"].T
    assert pu.max_rel_err(base, Y) > 10 * pu.TOL_OUT["bf16"]
    errs = {"Y": pu.max_rel_err(out["Y"], Y), "dX": pu.max_rel_err(out["dX"], g["dX"])}
    for k in g:
        if k != "dX":
            errs[k] = pu.rel_l2(out[k], g[k])
    print(cfg.name, kind, {k: f"{v:.2e}" for k, v in errs.items()})
    assert errs["Y"] <= pu.TOL_OUT["bf16"] and errs["dX"] <= pu.TOL_OUT["bf16"], errs
    for k in g:
        if k != "dX":
            assert errs[k] <= pu.TOL_GRAD["bf16"], errs
    return errs


KINDS = [l4q.L4Q_LORA_PLAIN, l4q.L4Q_LORA_QAT]


@pytest.mark.parametrize("kind", KINDS)
def test_exact_tiles(kind):
    cfg = synth.LayerConfig("variant_tiles", tokens=256, d_in=512, d_out=512, rank=16, alpha=32.0, bits=4,
                            group_size=128)
    check_variant(cfg, _inputs(cfg, 0), kind)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("rank,bits,group,signed", [(16, 4, 64, False), (8, 4, 32, True), (32, 3, 64, False),
                                                    (64, 3, 64, False)])
def test_ragged_tails(kind, rank, bits, group, signed):
    cfg = synth.LayerConfig(f"variant_ragged_r{rank}", tokens=300, d_in=832, d_out=392, rank=rank, alpha=32.0,
                            bits=bits, group_size=group, signed_grid=signed)
    check_variant(cfg, _inputs(cfg, 7), kind, grad_scale=0.25)


def test_qat_lora_with_clipped_weights():
    # a range shrunk to 80 % clips the extreme weights of every group: db and the bound terms of ds are non-zero
    cfg = synth.LayerConfig("variant_clipped", tokens=300, d_in=832, d_out=392, rank=16, alpha=32.0, bits=4,
                            group_size=64)
    arrays = _inputs(cfg, 9)
    arrays["s"] = (arrays["s"] * 0.8).astype(np.float32)
    out = run_variant(cfg, arrays, l4q.L4Q_LORA_QAT)
    assert np.abs(out["db"]).max() > 0
    check_variant(cfg, arrays, l4q.L4Q_LORA_QAT)


def test_qat_lora_wide_rows():
    # 20 groups per row: s and b reach the weight-tile kernel by TMA (the narrower cases above stage them by hand)
    cfg = synth.LayerConfig("variant_wide", tokens=200, d_in=1280, d_out=200, rank=16, alpha=32.0, bits=4,
                            group_size=64)
    arrays = _inputs(cfg, 15)
    arrays["s"] = (arrays["s"] * 0.9).astype(np.float32)
    check_variant(cfg, arrays, l4q.L4Q_LORA_QAT, grad_scale=0.5)


def test_plain_lora_takes_any_rank_up_to_64():
    cfg = synth.LayerConfig("variant_r12", tokens=200, d_in=320, d_out=264, rank=12, alpha=24.0, bits=4,
                            group_size=64)
    check_variant(cfg, _inputs(cfg, 3), l4q.L4Q_LORA_PLAIN)


@pytest.mark.parametrize("kind", KINDS)
def test_more_tiles_than_sms_and_token_split(kind):
    # forward: 3 x 56 tiles > 148 SMs; dA: 2 column tiles cut along 384 tokens; dB: 112 row tiles
    cfg = synth.LayerConfig("variant_persistent", tokens=384, d_in=320, d_out=14336, rank=16, alpha=32.0, bits=4,
                            group_size=64)
    check_variant(cfg, _inputs(cfg, 11), kind)


def test_long_token_axis():
    # 4096 tokens: the rank-side weight gradients run 64 K blocks, cut into slices over the idle SMs
    cfg = synth.LayerConfig("variant_tokens", tokens=4096, d_in=512, d_out=256, rank=16, alpha=32.0, bits=4,
                            group_size=128)
    check_variant(cfg, _inputs(cfg, 5), l4q.L4Q_LORA_PLAIN)


def test_argument_checks():
    gh.ensure_built()
    cfg = synth.LayerConfig("variant_args", tokens=128, d_in=256, d_out=256, rank=16, alpha=32.0, bits=4,
                            group_size=64)
    arrays = _inputs(cfg, 1)
    desc = l4q.make_desc(cfg)
    dev = l4q.to_device(cfg, arrays)
    outs = l4q.alloc_outputs(cfg)
    ws = l4q.alloc_lora_workspace(desc, l4q.L4Q_LORA_QAT, l4q.L4Q_OP_BWD)
    with pytest.raises(l4q.L4QError) as e:       # plain LoRA has no quantizer gradients
        l4q.l4q_lora_linear_bwd(desc, l4q.L4Q_LORA_PLAIN, dev["X"], dev["dY"], dev["W0"], dev["A"], dev["B"], None,
                                None, outs["dX"], outs["dA"], outs["dB"], outs["ds"], outs["db"], ws)
    assert e.value.status == 1
    with pytest.raises(l4q.L4QError) as e:       # QAT-LoRA needs s and b
        l4q.l4q_lora_linear_fwd(desc, l4q.L4Q_LORA_QAT, dev["X"], dev["W0"], dev["A"], dev["B"], None, None,
                                outs["Y"], ws)
    assert e.value.status == 1
    with pytest.raises(l4q.L4QError) as e:       # unknown kind
        l4q.l4q_lora_linear_fwd(desc, 7, dev["X"], dev["W0"], dev["A"], dev["B"], dev["s"], dev["b"], outs["Y"], ws)
    assert e.value.status == 1
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(l4q.L4QError) as e:
        l4q.l4q_lora_linear_fwd(desc, l4q.L4Q_LORA_PLAIN, dev["X"], dev["W0"], dev["A"], dev["B"], None, None,
                                outs["Y"], small)
    assert e.value.status == 3
    big = synth.LayerConfig("variant_r128", tokens=128, d_in=256, d_out=256, rank=128, alpha=32.0, bits=4,
                            group_size=64)
    assert l4q.l4q_lora_workspace_bytes(l4q.make_desc(big), l4q.L4Q_LORA_PLAIN, l4q.L4Q_OP_FWD) == 0
    # dX alone, and the parameter gradients alone
    l4q.l4q_lora_linear_bwd(desc, l4q.L4Q_LORA_QAT, dev["X"], dev["dY"], dev["W0"], dev["A"], dev["B"], dev["s"],
                            dev["b"], outs["dX"], None, None, None, None, ws)
    l4q.l4q_lora_linear_bwd(desc, l4q.L4Q_LORA_QAT, dev["X"], dev["dY"], dev["W0"], dev["A"], dev["B"], dev["s"],
                            dev["b"], None, outs["dA"], outs["dB"], outs["ds"], outs["db"], ws)
    l4q.l4q_check()
