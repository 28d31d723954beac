"""GPU parity of l4q_linear_infer (fully quantized inference from the packed export, Sec. 3.2 / App. F)
against the fp64 oracle: the kernel consumes exactly what l4q_pack_int wrote, so the test packs on the
GPU, checks the export against the oracle's (codes up to in-band ties, s16 / b16 bit-exact), and then
compares Y with the oracle's product over those same codes."""
import numpy as np
import pytest
import torch

from oracle import l4q_oracle as orc
from paper_2402_04902_b200 import binding as l4q
from paper_2402_04902_b200 import synth

import gpu_harness as gh
import parity_utils as pu

pytestmark = pytest.mark.gpu


def _run(cfg, seed):
    gh.ensure_built()
    arrays = synth.make_layer_inputs(cfg, seed=seed)
    d = l4q.to_device(cfg, arrays)
    desc = l4q.make_desc(cfg)
    pk = l4q.alloc_pack_outputs(cfg)
    l4q.l4q_pack_int(desc, d["W0"], d["A"], d["B"], d["s"], d["b"], pk["codes"], pk["s16"], pk["b16"])
    Y = gh.Guarded((cfg.tokens, cfg.d_out), torch.bfloat16)
    l4q.l4q_linear_infer(desc, d["X"], pk["codes"], pk["s16"], pk["b16"], Y.view)
    l4q.l4q_check()
    assert Y.intact(), "out-of-bounds write around Y"
    spec = pu.spec_of(cfg)
    a = pu.widen(arrays)
    codes = pk["codes"].cpu().numpy().view(np.uint32)
    w = orc.prequant(spec, orc.merge(spec, a["W0"], a["A"], a["B"]), a["s"], a["b"])
    res = pu.check_codes(orc.unpack_int(spec, codes, cfg.d_in), spec, w)
    assert res["out_of_band"] == 0, res
    s16, b16 = pk["s16"].cpu().numpy(), pk["b16"].cpu().numpy()
    Y_ref = orc.infer(spec, a["X"], codes, s16, b16, bf16_reference=True)
    err = pu.max_rel_err(Y.view.double().cpu().numpy(), Y_ref)
    print(cfg.name, "Y", f"{err:.2e}")
    assert err <= pu.TOL_OUT["bf16"], err
    return err


@pytest.mark.parametrize("tokens", [1, 2, 3, 4, 5, 64, 200])
@pytest.mark.parametrize("bits,group", [(4, 128), (3, 64), (4, 32), (3, 96)])
def test_infer_few_tokens(tokens, bits, group):
    # d_in = 1152 = 9 k-blocks of 128 = 36 x 32 = 12 x 96; d_out = 200 leaves a ragged 64-row tile
    cfg = synth.LayerConfig(f"infer_b{bits}_g{group}_t{tokens}", tokens=tokens, d_in=1152, d_out=200, rank=16,
                            alpha=32.0, bits=bits, group_size=group)
    _run(cfg, seed=41)


def test_infer_ragged_k_and_many_tiles():
    # d_in = 1184 = 9.25 k-blocks (last one mostly beyond the weight); 160 row tiles > 148 SMs
    cfg = synth.LayerConfig("infer_ragged", tokens=33, d_in=1184, d_out=10240, rank=8, alpha=16.0, bits=4,
                            group_size=32, signed_grid=True)
    _run(cfg, seed=42)


def test_infer_llama7b_mlp_up_batch_16():
    # full-size weight of the benchmark layer, a 16-token step (regime of Table 12)
    _run(synth.CONFIG3A.with_(name="infer_cfg3a_b16", tokens=16), seed=0)


def test_infer_llama7b_mlp_down_batch_64():
    # 11008 -> 4096: 86 k-steps on narrow tiles (32 weight rows per SM)
    _run(synth.CONFIG3B.with_(name="infer_cfg3b_b64", tokens=64), seed=0)


def test_infer_llama7b_attn_proj_batch_16():
    _run(synth.CONFIG2.with_(name="infer_cfg2_b16", tokens=16), seed=0)


@pytest.mark.parametrize("d_in,d_out,tokens,bits", [(4096, 1000, 1, 4), (4096, 1000, 4, 4), (11008, 520, 1, 4),
                                                    (11008, 520, 2, 4), (14336, 264, 1, 4), (4096, 392, 2, 3),
                                                    (11008, 392, 1, 3), (11008, 392, 3, 4)])
def test_infer_matrix_vector_shapes(d_in, d_out, tokens, bits):
    # one to four tokens on full-length rows (4096, 11008, 14336 values of k), output widths that leave a ragged
    # last tile, both bit widths: the matrix-vector kernel up to two tokens, the tensor-core kernel beyond
    cfg = synth.LayerConfig(f"infer_mv_{d_in}_{tokens}_{bits}", tokens=tokens, d_in=d_in, d_out=d_out, rank=8,
                            alpha=16.0, bits=bits, group_size=128 if bits == 4 else 64)
    _run(cfg, seed=5)


def test_infer_rejects_what_it_does_not_cover():
    gh.ensure_built()
    cfg = synth.LayerConfig("infer_bad_group", tokens=4, d_in=1040, d_out=64, rank=8, alpha=16.0, bits=4,
                            group_size=104)                                   # 104 % 32 != 0
    desc = l4q.make_desc(cfg)
    dummy = torch.zeros(4096, dtype=torch.int32, device="cuda")
    with pytest.raises(l4q.L4QError) as e:
        l4q.l4q_linear_infer(desc, dummy, dummy, dummy, dummy, dummy)
    assert e.value.status == 2
