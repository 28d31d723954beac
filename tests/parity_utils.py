"""Comparison helpers shared by the GPU parity tests (tolerances in one place).

Tolerances:
  * integer codes: bit-exact, except where the fp64 grid coordinate w lies
    within 1e-6 * max(1, |w|) of a rounding boundary k + 1/2; the number of such
    mismatches must not exceed 1e-6 of all elements; any other mismatch fails;
  * Y, dX: max_e |y - ref| / max(|ref|, rms(ref)) <= 2e-2 in bf16 (against the
    oracle's bf16-reference mode) and <= 1e-4 in the fp32 validation mode;
  * dA, dB, ds, db: relative L2 error <= 3e-2 in bf16, <= 1e-4 in fp32 mode.
"""
from __future__ import annotations

import math

import numpy as np

from oracle import l4q_oracle as orc

TOL_OUT = {"bf16": 2e-2, "f32": 1e-4}
TOL_GRAD = {"bf16": 3e-2, "f32": 1e-4}
CODE_BAND = 1e-6
CODE_FRACTION = 1e-6


def spec_of(cfg, grad_scale: float = 1.0) -> orc.L4QSpec:
    return orc.L4QSpec(rank=cfg.rank, alpha=cfg.alpha, bits=cfg.bits, group_size=cfg.group_size,
                       signed_grid=cfg.signed_grid, grad_scale=grad_scale)


def max_rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    if ref.size == 0:
        return 0.0
    rms = math.sqrt(float(np.mean(ref * ref)))
    den = np.maximum(np.abs(ref), rms if rms > 0 else 1.0)
    return float(np.max(np.abs(got - ref) / den))


def rel_l2(got: np.ndarray, ref: np.ndarray) -> float:
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    den = float(np.linalg.norm(ref))
    num = float(np.linalg.norm(got - ref))
    return num / den if den > 0 else num


def check_codes(got_u: np.ndarray, spec: orc.L4QSpec, w64: np.ndarray) -> dict:
    """Compare unsigned codes from the GPU with the oracle's, element by element.

    Returns {"mismatches", "out_of_band", "allowed"}; the caller asserts
    out_of_band == 0 and mismatches <= allowed."""
    qn, _ = orc.grid_bounds(spec)
    ref_u = (orc.quant_codes(spec, w64) - qn).astype(np.int64)
    got_u = np.asarray(got_u).astype(np.int64)
    bad = got_u != ref_u
    n_bad = int(bad.sum())
    out_of_band = 0
    if n_bad:
        wb = w64[bad]
        dist = np.abs(np.abs(wb - np.floor(wb)) - 0.5)          # distance to the nearest k + 1/2
        near = dist <= CODE_BAND * np.maximum(1.0, np.abs(wb))
        off_by_one = np.abs(got_u[bad] - ref_u[bad]) == 1
        out_of_band = int((~(near & off_by_one)).sum())
    return {"mismatches": n_bad, "out_of_band": out_of_band, "allowed": CODE_FRACTION * w64.size}


def widen(arrays: dict) -> dict:
    """float32 numpy inputs -> float64 (exact)."""
    return {k: np.asarray(v, dtype=np.float64) for k, v in arrays.items()}
