"""l4q_linear_fwd_static: the forward pass for callers that cannot allocate.

Some users of this library run where a device allocation is not an option: a
custom op inside a serving or training runtime whose allocator already owns the
GPU's free memory, or a loop that must never pay for cudaMalloc's device-wide
synchronisation.  For them the library carries a fixed 32 MiB scratch array and an
entry point that takes no workspace.  This test calls that entry point through
the C ABI and requires its output to equal l4q_linear_fwd's (same kernels, same
arithmetic, so the comparison is exact, well inside the 2e-2 / 1e-4 parity
tolerances) and to agree with the fp64 oracle within the bf16 forward tolerance,
on two calls in a row that share the array: the second call uses a
smaller, different layer, so anything it read from the first call's leftovers
would show.  Collected last on purpose (file name), and self-contained so that it
passes alone in a fresh process as well as after the other tests.
"""
import gc

import numpy as np
import pytest
import torch

from oracle import l4q_oracle as orc
from paper_2402_04902_b200 import binding as l4q
from paper_2402_04902_b200 import synth

import gpu_harness as gh
import parity_utils as pu

pytestmark = pytest.mark.gpu


def _run_both(cfg, seed):
    arrays = synth.make_layer_inputs(cfg, seed=seed)
    d = l4q.to_device(cfg, arrays)
    desc = l4q.make_desc(cfg)
    io = torch.bfloat16 if cfg.io_dtype == "bf16" else torch.float32
    y_ws = torch.full((cfg.tokens, cfg.d_out), float("nan"), dtype=io, device="cuda")
    y_static = torch.full((cfg.tokens, cfg.d_out), float("nan"), dtype=io, device="cuda")
    ws = l4q.alloc_workspace(desc, l4q.L4Q_OP_FWD)
    l4q.l4q_linear_fwd(desc, d["X"], d["W0"], d["A"], d["B"], d["s"], d["b"], y_ws, ws)
    gc.collect()                                                   # so that only the call below can move the counter
    torch.cuda.synchronize()
    mem_before = torch.cuda.memory_allocated()
    launches_before = l4q.l4q_launch_count()
    l4q.l4q_linear_fwd_static(desc, d["X"], d["W0"], d["A"], d["B"], d["s"], d["b"], y_static)
    l4q.l4q_check()
    assert l4q.l4q_launch_count() - launches_before == 2           # dequantize + GEMM, as in l4q_linear_fwd
    assert torch.cuda.memory_allocated() == mem_before             # nothing taken from torch's allocator
    assert not torch.isnan(y_static.float()).any()
    return y_ws, y_static


def _check_against_oracle(cfg, seed, y_static):
    """The entry point's own output against the fp64 oracle (Eq. 7-10, bf16 reference mode), not only against
    the other entry point: the same tolerance as every bf16 forward check, 2e-2.  The oracle takes its own
    codes except where the export of the same layer holds the other neighbour of a verified in-band tie."""
    arrays = synth.make_layer_inputs(cfg, seed=seed)
    spec = pu.spec_of(cfg)
    a = pu.widen(arrays)
    d = l4q.to_device(cfg, arrays)
    pk = l4q.alloc_pack_outputs(cfg)
    l4q.l4q_pack_int(l4q.make_desc(cfg), d["W0"], d["A"], d["B"], d["s"], d["b"], pk["codes"], pk["s16"], pk["b16"])
    l4q.l4q_check()
    qn, _ = orc.grid_bounds(spec)
    w = orc.prequant(spec, orc.merge(spec, a["W0"], a["A"], a["B"]), a["s"], a["b"])
    got_u = orc.unpack_int(spec, pk["codes"].cpu().numpy().view(np.uint32), cfg.d_in)
    res = pu.check_codes(got_u, spec, w)
    assert res["out_of_band"] == 0 and res["mismatches"] <= max(1.0, res["allowed"]), res
    codes = orc.quant_codes(spec, w)
    tie = (got_u + qn) != codes
    codes[tie] = (got_u + qn)[tie]
    Y = orc.forward(spec, a["X"], a["W0"], a["A"], a["B"], a["s"], a["b"], bf16_reference=True, codes=codes)
    err = pu.max_rel_err(y_static.double().cpu().numpy(), Y)
    assert err <= pu.TOL_OUT["bf16"], (cfg.name, err)


def test_static_forward_matches_workspace_forward_on_two_calls_in_a_row():
    gh.ensure_built()
    first = synth.LayerConfig("static_bf16_a", tokens=384, d_in=1024, d_out=768, rank=16, alpha=32.0, bits=4,
                              group_size=128)
    second = synth.LayerConfig("static_bf16_b", tokens=200, d_in=320, d_out=264, rank=8, alpha=16.0, bits=3,
                               group_size=64, signed_grid=True)
    for cfg, seed in ((first, 31), (second, 32)):
        y_ws, y_static = _run_both(cfg, seed)
        assert torch.equal(y_ws, y_static), cfg.name
        _check_against_oracle(cfg, seed, y_static)
    # the fp32 validation path shares the same array
    y_ws, y_static = _run_both(synth.CONFIG1, 33)
    assert torch.equal(y_ws, y_static)


def test_static_forward_rejects_weights_beyond_the_fixed_array():
    gh.ensure_built()
    too_big = synth.LayerConfig("static_too_big", tokens=8, d_in=4096, d_out=4104, rank=16, alpha=32.0, bits=4,
                                group_size=128)                   # 4104 x 4096 bf16 > 32 MiB
    assert too_big.d_in * too_big.d_out * 2 > l4q.L4Q_STATIC_SCRATCH_BYTES
    desc = l4q.make_desc(too_big)
    dummy = torch.zeros(64, dtype=torch.float32, device="cuda")     # never dereferenced: the size check comes first
    n0 = l4q.l4q_launch_count()
    with pytest.raises(l4q.L4QError) as e:
        l4q.l4q_linear_fwd_static(desc, dummy, dummy, dummy, dummy, dummy, dummy, dummy)
    assert e.value.status == 3                                       # L4Q_ERR_WORKSPACE
    assert l4q.l4q_launch_count() == n0
    exact_fit = too_big.with_(d_out=4096)
    assert exact_fit.d_in * exact_fit.d_out * 2 == l4q.L4Q_STATIC_SCRATCH_BYTES
