"""Runs the CUDA library on one synthetic layer and returns numpy results (test helper)."""
from __future__ import annotations

import numpy as np
import torch

from paper_2402_04902_b200 import binding as l4q
from paper_2402_04902_b200 import build as l4q_build

_CANARY = 1024  # elements of guard region on each side of every output


def ensure_built():
    l4q_build.build()
    return l4q.lib()


class Guarded:
    """Output tensor surrounded by NaN / sentinel guard regions, to catch
    out-of-bounds writes without a sanitizer."""

    def __init__(self, shape, dtype, device="cuda"):
        n = int(np.prod(shape))
        self.buf = torch.empty(n + 2 * _CANARY, dtype=dtype, device=device)
        self.sentinel = -7777 if not dtype.is_floating_point else float("nan")
        self.buf.fill_(self.sentinel)
        self.view = self.buf[_CANARY:_CANARY + n].view(*shape)

    def intact(self) -> bool:
        lo, hi = self.buf[:_CANARY], self.buf[-_CANARY:]
        if self.buf.dtype.is_floating_point:
            return bool(torch.isnan(lo).all() and torch.isnan(hi).all())
        return bool((lo == self.sentinel).all() and (hi == self.sentinel).all())


def run_layer(cfg, arrays, do_fwd=True, do_bwd=True, do_pack=False, grad_scale=1.0):
    """arrays: numpy dict from synth.make_layer_inputs. Returns dict of numpy outputs (float64 / ints)."""
    ensure_built()
    M = arrays["X"].shape[0] if "X" in arrays else cfg.tokens
    desc = l4q.make_desc(cfg, grad_scale=grad_scale, tokens=M)
    dev = l4q.to_device(cfg, arrays)
    io = torch.bfloat16 if cfg.io_dtype == "bf16" else torch.float32
    G = cfg.d_in // cfg.group_size
    out = {}
    guards = {}
    if do_fwd:
        ws = l4q.alloc_workspace(desc, l4q.L4Q_OP_FWD)
        guards["Y"] = Guarded((M, cfg.d_out), io)
        l4q.l4q_linear_fwd(desc, dev["X"], dev["W0"], dev["A"], dev["B"], dev["s"], dev["b"], guards["Y"].view, ws)
    if do_bwd:
        ws = l4q.alloc_workspace(desc, l4q.L4Q_OP_BWD)
        guards["dX"] = Guarded((M, cfg.d_in), io)
        guards["dA"] = Guarded((cfg.rank, cfg.d_in), torch.float32)
        guards["dB"] = Guarded((cfg.d_out, cfg.rank), torch.float32)
        guards["ds"] = Guarded((cfg.d_out, G), torch.float32)
        guards["db"] = Guarded((cfg.d_out, G), torch.float32)
        l4q.l4q_linear_bwd(desc, dev["X"], dev["dY"], dev["W0"], dev["A"], dev["B"], dev["s"], dev["b"],
                           guards["dX"].view, guards["dA"].view, guards["dB"].view, guards["ds"].view,
                           guards["db"].view, ws)
    if do_pack:
        guards["codes"] = Guarded((cfg.d_out, cfg.d_in * cfg.bits // 32), torch.int32)
        guards["s16"] = Guarded((cfg.d_out, G), torch.float16)
        guards["b16"] = Guarded((cfg.d_out, G), torch.float16)
        # with the optional scratch (the split operands are then built once); the calls elsewhere in the
        # tests pass none and cover the other path
        l4q.l4q_pack_int(desc, dev["W0"], dev["A"], dev["B"], dev["s"], dev["b"], guards["codes"].view,
                         guards["s16"].view, guards["b16"].view, l4q.alloc_workspace(desc, l4q.L4Q_OP_PACK))
    l4q.l4q_check()
    for k, g in guards.items():
        assert g.intact(), f"out-of-bounds write around {k}"
        v = g.view
        if k == "codes":
            out[k] = v.cpu().numpy().view(np.uint32)
        elif k in ("s16", "b16"):
            out[k] = v.cpu().numpy()
        else:
            out[k] = v.to(torch.float64).cpu().numpy()
    return out
