"""Plain fp64 CPU oracle of the L4Q quantization-aware LoRA linear layer.

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct
statement of what the CUDA library computes.  It shares no code with the CUDA
path, imports nothing from it, and must never be called by it.

Every function follows one passage of the paper (arXiv 2402.04902) in the
paper's order and notation; there is no blocking, fusion or reordering.
Matrix products use numpy's fp64 matmul as a library step.

Layout (row-major, tokens flattened; the paper writes column vectors,
``Y = W X``, this file writes the transposed, equivalent ``Y = X W^T``):

    X  [M, i]   activations            dY [M, o]   upstream gradient
    W0 [o, i]   frozen weight          A  [r, i], B [o, r]  LoRA factors
    s, b [o, i/g]  scale / offset of each group of g consecutive elements
                   of a weight row (groups run along d_in)

Readings taken where the paper is silent or needs a finite-precision rule:
  * the paper's constant "alpha" in Eq. 7 is ``gamma = alpha / rank`` here;
  * round() is round-half-to-even;
  * the integer grid is [Q_N, Q_P] = [-2^(n-1), 2^(n-1)-1] as in Eq. 3 when
    ``signed_grid`` is set, else the shifted twin [0, 2^n - 1];
  * the in-range test of the STE uses the *unrounded* w and is inclusive,
    as printed in App. A.1 / Eq. 13-14, widened by a guard band of
    ``mask_guard`` = 2^-10 of a quantization step on either side: a min/max
    initialisation puts the extreme element of every group exactly on a bound
    (w = Q_P up to the rounding of s), and Table 4 reports zero clipping for
    that initialisation, so an element on the bound must count as inside no
    matter which way the last bit of s was rounded;
  * dX = dY W_q is the textbook linear backward (the paper never prints it);
  * the packed export format (bit order, fp16 parameters) is this library's.

Pinned by tests/test_oracle_pins.py and tests/test_oracle_init_pins.py
against: B = 0 => merge == W0; grid membership; zero clipping under the
Asymm / L4Q_init initialisations (Table 4, "Initial" E_clip = 0.0); the LoRA
limits of Eq. 1-2; finite differences of the STE surrogate; a hand-worked
example; scalar brute force on tiny layers; pack/unpack round trips; the
printed gate of App. A.1 (guard band 0) away from the bounds.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class L4QSpec:
    """Hyper-parameters of one L4Q linear layer (Sec. 2.1, 2.2, 3.2)."""

    rank: int
    alpha: float
    bits: int
    group_size: int
    signed_grid: bool = False
    grad_scale: float = 1.0
    mask_guard: float = 2.0 ** -10    # guard band of the in-range test, in quantization steps

    @property
    def gamma(self) -> float:
        return float(self.alpha) / float(self.rank)


def grid_bounds(spec: L4QSpec) -> tuple[int, int]:
    """(Q_N, Q_P) of Eq. 3: signed [-2^(n-1), 2^(n-1)-1], or shifted to start at 0."""
    n = spec.bits
    if spec.signed_grid:
        return -(1 << (n - 1)), (1 << (n - 1)) - 1
    return 0, (1 << n) - 1


def _f64(x) -> np.ndarray:
    return np.asarray(x, dtype=np.float64)


def _expand_groups(p: np.ndarray, group_size: int) -> np.ndarray:
    """[o, G] per-group parameter -> [o, G*g], one value per weight element."""
    return np.repeat(p, group_size, axis=1)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp64 values to the nearest bfloat16 (8 significant bits, ties to
    even) and return them as fp64.  Normal range only (no subnormal/overflow
    handling: layer values are O(1e-3 .. 1e3))."""
    x = _f64(x)
    m, e = np.frexp(x)                    # x = m * 2^e, 0.5 <= |m| < 1
    return np.ldexp(np.rint(m * 256.0) / 256.0, e)


def merge(spec: L4QSpec, W0, A, B) -> np.ndarray:
    """Eq. 7: W_comb = W0 + gamma * B A."""
    return _f64(W0) + spec.gamma * (_f64(B) @ _f64(A))


def prequant(spec: L4QSpec, W_comb, s, b) -> np.ndarray:
    """w = (W_comb - b) / s, the unrounded grid coordinate (App. A.2, definition of w)."""
    g = spec.group_size
    return (_f64(W_comb) - _expand_groups(_f64(b), g)) / _expand_groups(_f64(s), g)


def quant_codes(spec: L4QSpec, w) -> np.ndarray:
    """Eq. 8: w~ = round(clamp(w, Q_N, Q_P)), integer-valued fp64."""
    qn, qp = grid_bounds(spec)
    return np.rint(np.minimum(np.maximum(_f64(w), qn), qp))


def dequant(spec: L4QSpec, w_tilde, s, b) -> np.ndarray:
    """Eq. 9: W_q = w~ * s + b."""
    g = spec.group_size
    return _f64(w_tilde) * _expand_groups(_f64(s), g) + _expand_groups(_f64(b), g)


def fake_quant_weight(spec: L4QSpec, W0, A, B, s, b, codes=None):
    """Eq. 7-9 in order.  Returns (w, w~, W_q).

    ``codes``: optional integer array taken as w~ instead of Eq. 8.  Where w sits
    on (or within rounding error of) a tie k + 1/2, both neighbours are correct
    results of round(); a caller that has checked another implementation's codes
    to be such neighbours passes them here so that everything downstream of the
    rounding decision is compared on the same decision.
    """
    w = prequant(spec, merge(spec, W0, A, B), s, b)
    wt = quant_codes(spec, w) if codes is None else _f64(codes)
    return w, wt, dequant(spec, wt, s, b)


def forward(spec: L4QSpec, X, W0, A, B, s, b, bf16_reference: bool = False, codes=None) -> np.ndarray:
    """Eq. 10: Y = X W_q^T.

    ``bf16_reference``: W_q is rounded to bf16 before the product and Y after
    it (what a bf16-operand, wide-accumulate GEMM sees); all sums stay fp64.
    """
    _, _, Wq = fake_quant_weight(spec, W0, A, B, s, b, codes)
    if bf16_reference:
        Wq = round_to_bf16(Wq)
    Y = _f64(X) @ Wq.T
    return round_to_bf16(Y) if bf16_reference else Y


def backward(spec: L4QSpec, X, dY, W0, A, B, s, b, bf16_reference: bool = False, codes=None) -> dict:
    """Backward of the layer; nothing is taken from the forward pass (App. E.2:
    the quantized weight is recomputed).

      dX = dY W_q                                   (textbook; implied by Eq. 10)
      G  = dL/dW_q = dY^T X                         (Eq. 11)
      m  = [Q_N - guard <= w <= Q_P + guard]        (App. A.1, STE of round.clamp; guard: see header)
      ds = sum_group G * {Q_N | w~ - w | Q_P}       (Eq. 5 and App. A.1, three cases)
      db = sum_group G * (1 - m)                    (Eq. 6 and App. A.1)
      dA = gamma * B^T (G * m)                      (Eq. 13 / App. A.2)
      dB = gamma * (G * m) A^T                      (Eq. 14 / App. A.2)
    """
    X, dY, A, B = _f64(X), _f64(dY), _f64(A), _f64(B)
    g = spec.group_size
    qn, qp = grid_bounds(spec)
    w, wt, Wq = fake_quant_weight(spec, W0, A, B, s, b, codes)

    Wq_mm = round_to_bf16(Wq) if bf16_reference else Wq
    dX = dY @ Wq_mm
    if bf16_reference:
        dX = round_to_bf16(dX)

    G = dY.T @ X                                            # Eq. 11, [o, i]
    in_range = (w >= qn - spec.mask_guard) & (w <= qp + spec.mask_guard)
    m = in_range.astype(np.float64)

    dWq_ds = np.where(in_range, wt - w, np.where(w < qn, float(qn), float(qp)))   # out of range: the violated bound
    dWq_db = 1.0 - m
    o, i = G.shape
    ds = spec.grad_scale * (G * dWq_ds).reshape(o, i // g, g).sum(axis=2)
    db = spec.grad_scale * (G * dWq_db).reshape(o, i // g, g).sum(axis=2)

    Gm = G * m
    dA = spec.gamma * (B.T @ Gm)
    dB = spec.gamma * (Gm @ A.T)
    return {"dX": dX, "dA": dA, "dB": dB, "ds": ds, "db": db}


def pack_int(spec: L4QSpec, W0, A, B, s, b):
    """Export of the fully quantized weight (Sec. 3.2: only w~, s, b are kept).

    The paper fixes no storage format; this library's is:
      u = w~ - Q_N  in [0, 2^n - 1]                 (unsigned code)
      row bitstream: code j occupies bits [j*n, (j+1)*n), least significant bit
      first, cut into little-endian 32-bit words -> codes[o, i*n/32] uint32
      s16 = fp16(s);  b16 = fp16(fp32(b + s*Q_N))   (offset of the unsigned code;
      formed in fp32, the precision s and b are trained in, then narrowed)
    so that W_q ~= u * s16 + b16.  Returns (codes uint32, s16 float16, b16 float16).
    """
    n = spec.bits
    qn, _ = grid_bounds(spec)
    _, wt, _ = fake_quant_weight(spec, W0, A, B, s, b)
    u = (wt - qn).astype(np.int64)
    o, i = u.shape
    if (i * n) % 32 != 0:
        raise ValueError("d_in * bits must be a multiple of 32")
    bits = ((u[:, :, None] >> np.arange(n, dtype=np.int64)) & 1).astype(np.uint8)   # [o, i, n], LSB first
    stream = bits.reshape(o, i * n)
    words = np.packbits(stream, axis=1, bitorder="little").view("<u4")
    s16 = _f64(s).astype(np.float16)
    b16 = (_f64(b) + _f64(s) * qn).astype(np.float32).astype(np.float16)
    return np.ascontiguousarray(words), s16, b16


def unpack_int(spec: L4QSpec, codes: np.ndarray, d_in: int) -> np.ndarray:
    """Inverse of the bitstream of :func:`pack_int`: uint32 words -> unsigned codes [o, d_in]."""
    n = spec.bits
    codes = np.ascontiguousarray(codes.astype("<u4"))
    o = codes.shape[0]
    stream = np.unpackbits(codes.view(np.uint8), axis=1, bitorder="little")[:, : d_in * n]
    bits = stream.reshape(o, d_in, n).astype(np.int64)
    return (bits << np.arange(n, dtype=np.int64)).sum(axis=2)


# ---------------------------------------------------------------------------
# Quantization-parameter initialisation (Sec. 3.3, Eq. 15; App. B) and the
# error sums of Table 4.
# ---------------------------------------------------------------------------

INIT_METHODS = ("lsq+", "symm", "asymm", "l4q")
S_FLOOR = 1e-8          # s > 0 is a precondition of Eq. 3; a constant group would give s = 0


def init_params(spec: L4QSpec, W, method: str):
    """s, b [o, i/g] of every group of the weight W [o, i], App. B, as printed for the
    signed grid [Q_N, Q_P] = [-2^(n-1), 2^(n-1) - 1]:

        LSQ+_init  s = max(|mu - 3 sigma|, |mu + 3 sigma|) / 2^(n-1),  b = 0
        Symm       s = max|W| / 2^(n-1),                               b = 0
        Asymm      s = (max W - min W) / (Q_P - Q_N),                  b = min W - s Q_N
        L4Q_init   s = max(|min W / Q_N|, |max W / Q_P|),              b = 0      (Eq. 15)

    mu, sigma: mean and (population) standard deviation of the group.  On the shifted grid
    [0, 2^n - 1] the same quantizer has b' = b + s Q_N (Q_N of the signed grid), which is
    what is returned when ``spec.signed_grid`` is False.  s is floored at S_FLOOR.
    """
    W = _f64(W)
    g, n = spec.group_size, spec.bits
    o, i = W.shape
    Wg = W.reshape(o, i // g, g)
    qn_s, qp_s = -(2 ** (n - 1)), 2 ** (n - 1) - 1
    lo, hi = Wg.min(axis=2), Wg.max(axis=2)
    b = np.zeros_like(lo)
    if method == "lsq+":
        mu, sigma = Wg.mean(axis=2), Wg.std(axis=2)
        s = np.maximum(np.abs(mu - 3.0 * sigma), np.abs(mu + 3.0 * sigma)) / 2.0 ** (n - 1)
    elif method == "symm":
        s = np.abs(Wg).max(axis=2) / 2.0 ** (n - 1)
    elif method == "asymm":
        s = (hi - lo) / float(qp_s - qn_s)
        s = np.maximum(s, S_FLOOR)
        b = lo - s * qn_s
    elif method == "l4q":
        s = np.maximum(np.abs(lo / qn_s), np.abs(hi / qp_s))
    else:
        raise ValueError(f"unknown initialisation {method!r}")
    s = np.maximum(s, S_FLOOR)
    if not spec.signed_grid:
        b = b + s * qn_s
    return s, b


def quant_error(spec: L4QSpec, W0, A, B, s, b):
    """(E_quant, E_clip) of Table 4 for the merged weight.

    The paper names them "sum of quantization errors" and "clipping errors caused by
    overflowed outliers" without a formula; the reading taken here:
        E_quant = sum over all weights of |W_comb - W_q|,
        E_clip  = the part of that sum that comes from weights outside the quantization
                  range, i.e. where the STE gate of App. A.1 is closed (same guard band).
    """
    w, _, W_q = fake_quant_weight(spec, W0, A, B, s, b)
    err = np.abs(merge(spec, W0, A, B) - W_q)
    qn, qp = grid_bounds(spec)
    clipped = (w < qn - spec.mask_guard) | (w > qp + spec.mask_guard)
    return float(err.sum()), float(err[clipped].sum())


# ---------------------------------------------------------------------------
# Fully quantized inference (Sec. 3.2, App. F): only the export is kept.
# ---------------------------------------------------------------------------

def infer(spec: L4QSpec, X, codes: np.ndarray, s16, b16, bf16_reference: bool = False) -> np.ndarray:
    """Y = X W_q^T with the weight rebuilt from the export of :func:`pack_int`:
    W_q[o, j] = u[o, j] * s16[o, j // g] + b16[o, j // g]   (Eq. 9 on the unsigned code).

    ``bf16_reference``: W_q is rounded to bf16 before the product and Y after it, as a
    bf16 tensor-core path does (fp32 accumulation is taken as exact here).
    """
    X = _f64(X)
    u = _f64(unpack_int(spec, codes, X.shape[1]))
    g = spec.group_size
    W_q = u * _expand_groups(_f64(s16), g) + _expand_groups(_f64(b16), g)
    if bf16_reference:
        W_q = round_to_bf16(W_q)
    Y = X @ W_q.T
    return round_to_bf16(Y) if bf16_reference else Y


# ---------------------------------------------------------------------------
# Optimizer step for the trainable parameters A, B, s, b (App. D: AdamW with weight decay 0.01).
# ---------------------------------------------------------------------------

def adamw_step(param, grad, m, v, step: int, lr: float, beta1: float = 0.9, beta2: float = 0.999,
               eps: float = 1e-8, weight_decay: float = 0.01):
    """One AdamW update (decoupled weight decay), the published algorithm step by step:
        p  <- p - lr * wd * p
        m  <- beta1 m + (1 - beta1) g            v <- beta2 v + (1 - beta2) g^2
        mh <- m / (1 - beta1^t)                  vh <- v / (1 - beta2^t)
        p  <- p - lr * mh / (sqrt(vh) + eps)
    ``step`` t counts from 1.  Returns (param, m, v) as new fp64 arrays."""
    p, g, m, v = _f64(param), _f64(grad), _f64(m), _f64(v)
    p = p - lr * weight_decay * p
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    mh = m / (1.0 - beta1 ** step)
    vh = v / (1.0 - beta2 ** step)
    p = p - lr * mh / (np.sqrt(vh) + eps)
    return p, m, v


# ---------------------------------------------------------------------------
# The two layers L4Q is set against (Sec. 2.1 and 3.1): plain LoRA and QAT-LoRA, which
# keeps the quantized frozen weight and the high-precision LoRA path apart.
# ---------------------------------------------------------------------------

def lora_forward(spec: L4QSpec, X, W0, A, B, bf16_reference: bool = False) -> np.ndarray:
    """Eq. 1: Y = X W0^T + gamma (X A^T) B^T  (X~ = X A^T is the input of B)."""
    X = _f64(X)
    Xt = X @ _f64(A).T
    Y = X @ _f64(W0).T + spec.gamma * (Xt @ _f64(B).T)
    return round_to_bf16(Y) if bf16_reference else Y


def lora_backward(spec: L4QSpec, X, dY, W0, A, B, bf16_reference: bool = False) -> dict:
    """Eq. 2 in this file's layout, and the input gradient of Eq. 1:
        dA = gamma (dY B)^T X         dB = gamma dY^T X~,  X~ = X A^T
        dX = dY W0 + gamma (dY B) A
    """
    X, dY, A, B = _f64(X), _f64(dY), _f64(A), _f64(B)
    dYt = dY @ B                                    # gradient at the output of A, [M, r]
    Xt = X @ A.T
    dX = dY @ _f64(W0) + spec.gamma * (dYt @ A)
    if bf16_reference:
        dX = round_to_bf16(dX)
    return {"dX": dX, "dA": spec.gamma * (dYt.T @ X), "dB": spec.gamma * (dY.T @ Xt)}


def qat_lora_forward(spec: L4QSpec, X, W0, A, B, s, b, bf16_reference: bool = False, codes=None) -> np.ndarray:
    """QAT-LoRA (Sec. 3.1): the frozen weight alone goes through the quantizer of Eq. 3 / Eq. 8-9
    and the LoRA path of Eq. 1 is added in high precision:
        Y = X Q(W0)^T + gamma (X A^T) B^T.
    """
    X = _f64(X)
    zero_B = np.zeros((np.shape(W0)[0], spec.rank))
    _, _, Wq = fake_quant_weight(spec, W0, A, zero_B, s, b, codes)
    if bf16_reference:
        Wq = round_to_bf16(Wq)
    Y = X @ Wq.T + spec.gamma * ((X @ _f64(A).T) @ _f64(B).T)
    return round_to_bf16(Y) if bf16_reference else Y


def qat_lora_backward(spec: L4QSpec, X, dY, W0, A, B, s, b, bf16_reference: bool = False, codes=None) -> dict:
    """Backward of QAT-LoRA.  The LoRA factors get the LoRA gradients of Eq. 2, the quantizer gets
    the LSQ gradients of Eq. 5-6 from the full weight gradient G = dY^T X (the cost Sec. 3.1 points
    out), with w = (W0 - b) / s: the two sets of parameters do not see each other.
        dX = dY Q(W0) + gamma (dY B) A
    """
    X, dY, A, B = _f64(X), _f64(dY), _f64(A), _f64(B)
    g = spec.group_size
    qn, qp = grid_bounds(spec)
    zero_B = np.zeros((np.shape(W0)[0], spec.rank))
    w, wt, Wq = fake_quant_weight(spec, W0, A, zero_B, s, b, codes)
    if bf16_reference:
        Wq = round_to_bf16(Wq)
    dYt = dY @ B
    dX = dY @ Wq + spec.gamma * (dYt @ A)
    if bf16_reference:
        dX = round_to_bf16(dX)
    G = dY.T @ X
    in_range = (w >= qn - spec.mask_guard) & (w <= qp + spec.mask_guard)
    dWq_ds = np.where(in_range, wt - w, np.where(w < qn, float(qn), float(qp)))
    o, i = G.shape
    ds = spec.grad_scale * (G * dWq_ds).reshape(o, i // g, g).sum(axis=2)
    db = spec.grad_scale * (G * (1.0 - in_range)).reshape(o, i // g, g).sum(axis=2)
    return {"dX": dX, "dA": spec.gamma * (dYt.T @ X), "dB": spec.gamma * (dY.T @ (X @ A.T)), "ds": ds, "db": db}
