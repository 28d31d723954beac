"""Pins of the fp64 oracle against what the paper and the mathematics fix.

Nothing here compares the oracle with itself: every expected value is a
hand-worked number, a closed form, an invariant, a special case that reduces
to a textbook routine written out in the test, a finite difference, or a
scalar brute force.
"""
import json
import os

import numpy as np
import pytest

from oracle import l4q_oracle as orc
from oracle.l4q_oracle import L4QSpec

HERE = os.path.dirname(os.path.abspath(__file__))


def _layer(rng, o=6, i=16, r=2, M=5, g=4, bits=4, signed=False, alpha=4.0, bscale=0.05, spread=1.0):
    """Small random layer with a min/max grid per group widened by `spread`."""
    spec = L4QSpec(rank=r, alpha=alpha, bits=bits, group_size=g, signed_grid=signed)
    W0 = rng.normal(0, 0.3, (o, i))
    A = rng.uniform(-0.5, 0.5, (r, i))
    B = rng.normal(0, bscale, (o, r))
    X = rng.normal(0, 1, (M, i))
    dY = rng.normal(0, 1, (M, o))
    Wg = W0.reshape(o, i // g, g)
    lo, hi = Wg.min(2), Wg.max(2)
    qn, qp = orc.grid_bounds(spec)
    s = spread * (hi - lo) / (qp - qn)
    b = lo - s * qn
    return spec, X, dY, W0, A, B, s, b


# --------------------------------------------------------------------------
# hand-worked example (tests/golden/hand_example.json)
# --------------------------------------------------------------------------

def test_hand_worked_example():
    ex = json.load(open(os.path.join(HERE, "golden", "hand_example.json")))
    spec = L4QSpec(**ex["spec"])
    a = {k: np.array(ex[k], dtype=np.float64) for k in ("W0", "A", "B", "s", "b", "X", "dY")}
    e = {k: np.array(v, dtype=np.float64) for k, v in ex["expected"].items()}
    Wc = orc.merge(spec, a["W0"], a["A"], a["B"])
    w, wt, Wq = orc.fake_quant_weight(spec, a["W0"], a["A"], a["B"], a["s"], a["b"])
    tol = dict(rtol=0, atol=1e-12)
    np.testing.assert_allclose(Wc, e["W_comb"], **tol)
    np.testing.assert_allclose(w, e["w"], **tol)
    np.testing.assert_array_equal(wt, e["w_tilde"])
    np.testing.assert_allclose(Wq, e["W_q"], **tol)
    Y = orc.forward(spec, a["X"], a["W0"], a["A"], a["B"], a["s"], a["b"])
    np.testing.assert_allclose(Y, e["Y"], **tol)
    g = orc.backward(spec, a["X"], a["dY"], a["W0"], a["A"], a["B"], a["s"], a["b"])
    for k in ("dX", "ds", "db", "dA", "dB"):
        np.testing.assert_allclose(g[k], e[k], **tol, err_msg=k)
    # unsigned export codes: u = w~ - Q_N
    qn, _ = orc.grid_bounds(spec)
    np.testing.assert_array_equal(wt - qn, e["unsigned_codes"])


def test_round_half_to_even_and_clamp_before_round():
    # exact binary inputs: b = 0.25, s = 0.5, B = 0, signed 3-bit grid [-4, 3]
    spec = L4QSpec(rank=1, alpha=1.0, bits=3, group_size=8, signed_grid=True)
    w_target = np.array([[0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, -4.5]])
    W0 = 0.25 + 0.5 * w_target
    A = np.zeros((1, 8)); B = np.zeros((1, 1))
    s = np.array([[0.5]]); b = np.array([[0.25]])
    w, wt, _ = orc.fake_quant_weight(spec, W0, A, B, s, b)
    np.testing.assert_array_equal(w, w_target)
    # ties go to the even integer; 3.5 and -4.5 are clamped to 3 and -4 first
    np.testing.assert_array_equal(wt, [[0.0, 2.0, 2.0, -0.0, -2.0, -2.0, 3.0, -4.0]])


# --------------------------------------------------------------------------
# merge (Eq. 7)
# --------------------------------------------------------------------------

def test_merge_with_zero_B_is_W0_bit_for_bit():
    rng = np.random.default_rng(1)
    spec, X, dY, W0, A, B, s, b = _layer(rng)
    Wc = orc.merge(spec, W0, A, np.zeros_like(B))
    assert np.array_equal(Wc, W0)


def test_merge_rank_one_by_scalar_loops():
    rng = np.random.default_rng(2)
    spec, X, dY, W0, A, B, s, b = _layer(rng, r=1, alpha=3.0)
    Wc = orc.merge(spec, W0, A, B)
    for oo in range(W0.shape[0]):
        for j in range(W0.shape[1]):
            assert Wc[oo, j] == pytest.approx(W0[oo, j] + 3.0 * B[oo, 0] * A[0, j], abs=1e-15)


def test_merge_operand_order_not_transposed():
    # non-square case where B A has only one valid orientation, checked by loops
    rng = np.random.default_rng(3)
    spec = L4QSpec(rank=3, alpha=6.0, bits=4, group_size=4)
    W0 = rng.normal(size=(2, 8)); A = rng.normal(size=(3, 8)); B = rng.normal(size=(2, 3))
    Wc = orc.merge(spec, W0, A, B)
    ref = np.array([[W0[o, j] + 2.0 * sum(B[o, k] * A[k, j] for k in range(3)) for j in range(8)]
                    for o in range(2)])
    np.testing.assert_allclose(Wc, ref, rtol=0, atol=1e-14)


# --------------------------------------------------------------------------
# quantizer (Eq. 3, 8, 9)
# --------------------------------------------------------------------------

@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("signed", [False, True])
def test_grid_bounds(bits, signed):
    qn, qp = orc.grid_bounds(L4QSpec(1, 1.0, bits, 4, signed))
    assert qp - qn == 2 ** bits - 1
    assert qn == (-(2 ** (bits - 1)) if signed else 0)


@pytest.mark.parametrize("bits,signed", [(3, False), (4, False), (4, True)])
def test_dequantized_values_lie_on_group_grid(bits, signed):
    rng = np.random.default_rng(4)
    spec, X, dY, W0, A, B, s, b = _layer(rng, o=8, i=32, g=8, bits=bits, signed=signed, spread=0.8)
    w, wt, Wq = orc.fake_quant_weight(spec, W0, A, B, s, b)
    qn, qp = orc.grid_bounds(spec)
    assert np.array_equal(wt, np.round(wt))
    assert wt.min() >= qn and wt.max() <= qp
    g = spec.group_size
    for oo in range(8):
        for k in range(32 // g):
            vals = Wq[oo, k * g:(k + 1) * g]
            steps = (vals - b[oo, k]) / s[oo, k]
            np.testing.assert_allclose(steps, np.round(steps), atol=1e-9)
            assert len(np.unique(np.round(steps))) <= 2 ** bits
    # nearest-grid-point property inside the range: |w - w~| <= 1/2
    inside = (w >= qn) & (w <= qp)
    assert np.all(np.abs(w - wt)[inside] <= 0.5 + 1e-12)
    # outside the range the code is the violated bound
    assert np.all(wt[w < qn] == qn) and np.all(wt[w > qp] == qp)
    assert (w < qn).any() and (w > qp).any()      # spread=0.8 really clips


@pytest.mark.parametrize("signed", [False, True])
def test_asymm_init_has_zero_clipping_and_uses_both_ends(signed):
    """Table 4, column "Initial": E_clip = 0.0 under the min/max (Asymm) init."""
    rng = np.random.default_rng(5)
    spec, X, dY, W0, A, B, s, b = _layer(rng, o=8, i=32, g=8, signed=signed)
    B0 = np.zeros_like(B)
    w, wt, Wq = orc.fake_quant_weight(spec, W0, A, B0, s, b)
    qn, qp = orc.grid_bounds(spec)
    unclamped = np.rint(w)
    assert np.array_equal(unclamped, wt)                               # clamp never acted
    clip_err = np.abs(np.clip(w, qn, qp) - w).sum()
    assert clip_err < 1e-9
    wg = wt.reshape(8, 4, 8)
    assert np.all(wg.min(2) == qn) and np.all(wg.max(2) == qp)


def test_l4q_init_has_zero_clipping():
    """Eq. 15: s = max(|min/Q_N|, |max/Q_P|), b = 0 covers both extremes (Table 4, E_clip = 0.0)."""
    rng = np.random.default_rng(6)
    spec = L4QSpec(rank=2, alpha=4.0, bits=4, group_size=8, signed_grid=True)
    W0 = rng.normal(0, 0.3, (8, 32))
    Wg = W0.reshape(8, 4, 8)
    qn, qp = orc.grid_bounds(spec)
    s = np.maximum(np.abs(Wg.min(2) / qn), np.abs(Wg.max(2) / qp))
    b = np.zeros_like(s)
    A = rng.normal(size=(2, 32)); B = np.zeros((8, 2))
    w, wt, Wq = orc.fake_quant_weight(spec, W0, A, B, s, b)
    assert np.all((w >= qn - 1e-12) & (w <= qp + 1e-12))
    assert np.array_equal(np.rint(w), wt)
    assert np.abs(Wq - W0).max() <= 0.5 * s.max() + 1e-12


# --------------------------------------------------------------------------
# forward / dX (Eq. 10 and its textbook backward); LoRA limit (Eq. 1)
# --------------------------------------------------------------------------

def test_forward_and_dx_are_plain_products_of_Wq():
    rng = np.random.default_rng(7)
    spec, X, dY, W0, A, B, s, b = _layer(rng, o=5, i=12, g=4, M=3, spread=0.7)
    _, _, Wq = orc.fake_quant_weight(spec, W0, A, B, s, b)
    Y = orc.forward(spec, X, W0, A, B, s, b)
    dX = orc.backward(spec, X, dY, W0, A, B, s, b)["dX"]
    for t in range(3):
        for oo in range(5):
            assert Y[t, oo] == pytest.approx(sum(X[t, j] * Wq[oo, j] for j in range(12)), abs=1e-12)
        for j in range(12):
            assert dX[t, j] == pytest.approx(sum(dY[t, oo] * Wq[oo, j] for oo in range(5)), abs=1e-12)


def test_fine_grid_limit_is_lora_forward_and_backward():
    """With a very fine grid that clips nothing, Eq. 10 tends to Eq. 1 and
    Eq. 13-14 reduce exactly to Eq. 2 (mask == 1)."""
    rng = np.random.default_rng(8)
    o, i, r, M, g = 6, 16, 2, 5, 4
    spec = L4QSpec(rank=r, alpha=4.0, bits=8, group_size=g, signed_grid=True)
    W0 = rng.normal(0, 0.3, (o, i)); A = rng.uniform(-.5, .5, (r, i)); B = rng.normal(0, .05, (o, r))
    X = rng.normal(size=(M, i)); dY = rng.normal(size=(M, o))
    s = np.full((o, i // g), 2.0 / 127 / 1.0)        # range [-128 s, 127 s] ~ [-2, 2] covers all of W_comb
    b = np.zeros_like(s)
    gamma = spec.gamma
    Y = orc.forward(spec, X, W0, A, B, s, b)
    Y_lora = X @ W0.T + gamma * (X @ A.T) @ B.T                       # Eq. 1
    assert np.abs(Y - Y_lora).max() <= 0.5 * s.max() * np.abs(X).sum(1).max() + 1e-12
    grads = orc.backward(spec, X, dY, W0, A, B, s, b)
    Xt = X @ A.T                                                      # X~ = A X
    dA_lora = gamma * (dY @ B).T @ X                                  # Eq. 2
    dB_lora = gamma * dY.T @ Xt
    np.testing.assert_allclose(grads["dA"], dA_lora, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(grads["dB"], dB_lora, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(grads["db"], 0.0, atol=0)              # nothing outside the range
    dX_lora = dY @ (W0 + gamma * B @ A)
    assert np.abs(grads["dX"] - dX_lora).max() <= 0.5 * s.max() * np.abs(dY).sum(1).max() + 1e-12


# --------------------------------------------------------------------------
# gradients: finite differences of the STE surrogate and of the true forward
# --------------------------------------------------------------------------

def _surrogate_loss(spec, X, R, W0, A, B, s, b, frozen_c):
    """Loss sum(Y * R) with round() replaced by identity + a frozen residual
    (the straight-through estimator of App. A.1), written independently of the oracle."""
    qn, qp = orc.grid_bounds(spec)
    g = spec.group_size
    Wc = W0 + (spec.alpha / spec.rank) * B @ A
    se, be = np.repeat(s, g, 1), np.repeat(b, g, 1)
    w = (Wc - be) / se
    Wq = (np.clip(w, qn, qp) + frozen_c) * se + be
    return float(((X @ Wq.T) * R).sum())


def _fd(f, x, idx, h):
    xp = x.copy(); xp[idx] += h
    xm = x.copy(); xm[idx] -= h
    return (f(xp) - f(xm)) / (2 * h)


@pytest.mark.parametrize("signed", [False, True])
def test_all_parameter_gradients_match_fd_of_ste_surrogate(signed):
    rng = np.random.default_rng(9)
    spec, X, R, W0, A, B, s, b = _layer(rng, o=4, i=8, r=2, M=3, g=4, bits=3, signed=signed, spread=0.75)
    qn, qp = orc.grid_bounds(spec)
    w, wt, _ = orc.fake_quant_weight(spec, W0, A, B, s, b)
    # stay away from the kinks of clamp so that central differences are exact to O(h^2)
    assert np.abs(w - qn).min() > 1e-3 and np.abs(w - qp).min() > 1e-3
    assert ((w < qn) | (w > qp)).any() and ((w >= qn) & (w <= qp)).any()
    c = wt - np.clip(w, qn, qp)
    grads = orc.backward(spec, X, R, W0, A, B, s, b)
    h = 1e-6
    for name, arr in (("ds", s), ("db", b), ("dA", A), ("dB", B)):
        for idx in np.ndindex(arr.shape):
            def f(v, name=name):
                kw = dict(W0=W0, A=A, B=B, s=s, b=b)
                kw[{"ds": "s", "db": "b", "dA": "A", "dB": "B"}[name]] = v
                return _surrogate_loss(spec, X, R, frozen_c=c, **kw)
            fd = _fd(f, arr, idx, h)
            assert grads[name][idx] == pytest.approx(fd, rel=1e-6, abs=1e-6), (name, idx)


def test_true_fd_of_quantized_forward_vs_lsq_form():
    """Away from rounding boundaries the codes are locally constant, so the true
    derivative of the quantized forward w.r.t. s is sum(G * w~) and w.r.t. b is
    sum(G); the LSQ closed form differs from it by exactly -sum_{in range} G * w
    (resp. -sum_{in range} G).  Ties forward(), G and w of the oracle together."""
    rng = np.random.default_rng(10)
    spec, X, R, W0, A, B, s, b = _layer(rng, o=4, i=8, r=2, M=3, g=4, bits=3, spread=0.75)
    qn, qp = orc.grid_bounds(spec)
    w, wt, _ = orc.fake_quant_weight(spec, W0, A, B, s, b)
    assert np.abs((w - np.floor(w)) - 0.5).min() > 1e-3            # no element near a rounding boundary
    grads = orc.backward(spec, X, R, W0, A, B, s, b)
    G = R.T @ X
    inr = (w >= qn) & (w <= qp)
    loss = lambda s_, b_: float((orc.forward(spec, X, W0, A, B, s_, b_) * R).sum())
    h = 1e-7
    for idx in np.ndindex(s.shape):
        sl = slice(idx[1] * 4, idx[1] * 4 + 4)
        true_ds = _fd(lambda v: loss(v, b), s, idx, h)
        true_db = _fd(lambda v: loss(s, v), b, idx, h)
        assert true_ds == pytest.approx((G[idx[0], sl] * wt[idx[0], sl]).sum(), rel=1e-5, abs=1e-5)
        assert true_db == pytest.approx(G[idx[0], sl].sum(), rel=1e-5, abs=1e-5)
        gap_s = (G[idx[0], sl] * w[idx[0], sl] * inr[idx[0], sl]).sum()
        gap_b = (G[idx[0], sl] * inr[idx[0], sl]).sum()
        assert grads["ds"][idx] == pytest.approx(true_ds - gap_s, rel=1e-5, abs=1e-5)
        assert grads["db"][idx] == pytest.approx(true_db - gap_b, rel=1e-5, abs=1e-5)


def test_ste_gate_blocks_lora_gradient_outside_range_and_is_inclusive():
    """Eq. 13-14: gradient flows to A, B only where Q_N <= w <= Q_P (inclusive);
    db collects exactly the complement (Eq. 6)."""
    spec = L4QSpec(rank=1, alpha=1.0, bits=2, group_size=4)          # unsigned grid [0, 3]
    s = np.array([[1.0]]); b = np.array([[0.0]])
    # w = W_comb: one below, exact lower bound, exact upper bound, one above
    W0 = np.array([[-0.25, 0.0, 3.0, 3.25]])
    A = np.array([[1.0, 2.0, 3.0, 4.0]]); B = np.array([[0.0]])
    X = np.eye(4); dY = np.array([[1.0], [10.0], [100.0], [1000.0]])  # G = [1, 10, 100, 1000]
    g = orc.backward(spec, X, dY, W0, A, B, s, b)
    np.testing.assert_array_equal(g["dA"], [[0.0, 0.0, 0.0, 0.0]])   # B = 0
    assert g["dB"][0, 0] == 10.0 * 2.0 + 100.0 * 3.0                 # only the two in-range columns
    assert g["db"][0, 0] == 1.0 + 1000.0
    # ds: below -> Q_N = 0, in range -> w~ - w = 0, above -> Q_P = 3
    assert g["ds"][0, 0] == 1.0 * 0 + 1000.0 * 3
    # 3.25 would round to 3 (= Q_P) but is outside the range: mask uses the unrounded w
    B1 = np.array([[1.0]])
    W0b = W0 - A                                                       # so that W_comb is unchanged
    g2 = orc.backward(spec, X, dY, W0b, A, B1, s, b)
    np.testing.assert_array_equal(g2["dA"], [[0.0, 10.0, 100.0, 0.0]])


def test_backward_is_linear_in_dY_and_additive_over_token_shards():
    rng = np.random.default_rng(11)
    spec, X, dY, W0, A, B, s, b = _layer(rng, o=6, i=16, M=8, spread=0.8)
    dY2 = rng.normal(size=dY.shape)
    g1 = orc.backward(spec, X, dY, W0, A, B, s, b)
    g2 = orc.backward(spec, X, dY2, W0, A, B, s, b)
    g12 = orc.backward(spec, X, 2.0 * dY - 3.0 * dY2, W0, A, B, s, b)
    for k in g1:
        np.testing.assert_allclose(g12[k], 2.0 * g1[k] - 3.0 * g2[k], rtol=1e-11, atol=1e-11)
    ga = orc.backward(spec, X[:3], dY[:3], W0, A, B, s, b)
    gb = orc.backward(spec, X[3:], dY[3:], W0, A, B, s, b)
    for k in ("dA", "dB", "ds", "db"):
        np.testing.assert_allclose(ga[k] + gb[k], g1[k], rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(np.vstack([ga["dX"], gb["dX"]]), g1["dX"], rtol=1e-12, atol=1e-12)


def test_signed_and_unsigned_grids_are_one_reparametrisation():
    """u = w~ - Q_N, b_u = b_s + s Q_N: same W_q, Y, dX, dA, dB; db equal; ds_u = ds_s - Q_N db_s."""
    rng = np.random.default_rng(12)
    spec_s, X, dY, W0, A, B, s, b_s = _layer(rng, o=6, i=16, signed=True, spread=0.8)
    spec_u = L4QSpec(spec_s.rank, spec_s.alpha, spec_s.bits, spec_s.group_size, signed_grid=False)
    qn, _ = orc.grid_bounds(spec_s)
    b_u = b_s + s * qn
    np.testing.assert_allclose(orc.forward(spec_s, X, W0, A, B, s, b_s),
                               orc.forward(spec_u, X, W0, A, B, s, b_u), rtol=1e-12, atol=1e-12)
    gs = orc.backward(spec_s, X, dY, W0, A, B, s, b_s)
    gu = orc.backward(spec_u, X, dY, W0, A, B, s, b_u)
    for k in ("dX", "dA", "dB", "db"):
        np.testing.assert_allclose(gs[k], gu[k], rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(gu["ds"], gs["ds"] - qn * gs["db"], rtol=1e-9, atol=1e-9)


def test_grad_scale_multiplies_only_ds_db():
    rng = np.random.default_rng(13)
    spec, X, dY, W0, A, B, s, b = _layer(rng, spread=0.8)
    spec2 = L4QSpec(spec.rank, spec.alpha, spec.bits, spec.group_size, spec.signed_grid, grad_scale=0.25)
    g1 = orc.backward(spec, X, dY, W0, A, B, s, b)
    g2 = orc.backward(spec2, X, dY, W0, A, B, s, b)
    for k in ("dX", "dA", "dB"):
        np.testing.assert_array_equal(g1[k], g2[k])
    for k in ("ds", "db"):
        np.testing.assert_allclose(g2[k], 0.25 * g1[k], rtol=1e-15)


# --------------------------------------------------------------------------
# pack (export of the fully quantized weight)
# --------------------------------------------------------------------------

@pytest.mark.parametrize("bits,signed", [(3, False), (4, False), (3, True), (4, True)])
def test_pack_bitstream_by_big_integer_brute_force(bits, signed):
    rng = np.random.default_rng(14)
    spec, X, dY, W0, A, B, s, b = _layer(rng, o=3, i=64, g=32, bits=bits, signed=signed, spread=0.9)
    codes, s16, b16 = orc.pack_int(spec, W0, A, B, s, b)
    _, wt, Wq = orc.fake_quant_weight(spec, W0, A, B, s, b)
    qn, _ = orc.grid_bounds(spec)
    assert codes.dtype == np.uint32 and codes.shape == (3, 64 * bits // 32)
    for oo in range(3):
        big = 0
        for j in range(64):
            big |= int(wt[oo, j] - qn) << (j * bits)
        for k in range(codes.shape[1]):
            assert int(codes[oo, k]) == (big >> (32 * k)) & 0xFFFFFFFF
    u = orc.unpack_int(spec, codes, 64)
    np.testing.assert_array_equal(u, wt - qn)
    # dequantising the export reproduces W_q up to the fp16 rounding of s and b
    se = np.repeat(s16.astype(np.float64), 32, 1); be = np.repeat(b16.astype(np.float64), 32, 1)
    err = np.abs(u * se + be - Wq)
    bound = (2 ** bits) * np.abs(s).max() * 2.0 ** -11 + np.abs(b + s * qn).max() * 2.0 ** -11 + 1e-7
    assert err.max() <= bound
    assert s16.dtype == np.float16 and b16.dtype == np.float16


def test_pack_three_bit_codes_straddle_words():
    """u_j = j mod 8 for 32 codes -> 96 bits -> 3 words, checked against a literal bit loop."""
    spec = L4QSpec(rank=1, alpha=1.0, bits=3, group_size=32)
    u = (np.arange(32) % 8).astype(np.float64)[None, :]
    s = np.array([[1.0]]); b = np.array([[0.0]])
    codes, _, _ = orc.pack_int(spec, u, np.zeros((1, 32)), np.zeros((1, 1)), s, b)
    bits = []
    for j in range(32):
        for k in range(3):
            bits.append((int(u[0, j]) >> k) & 1)
    words = [sum(bits[32 * w + t] << t for t in range(32)) for w in range(3)]
    assert [int(x) for x in codes[0]] == words
    assert words[0] == 0b10_001_000_111_110_101_100_011_010_001_000   # codes 0..9 whole, low 2 bits of code 10


def test_round_to_bf16():
    x = np.array([1.0, 1.00390625, 1.01171875, -3.1415926, 1e-3, 0.0])
    r = orc.round_to_bf16(x)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 ties to 1 + 2^-6
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.015625 and r[5] == 0.0
    import torch
    t = torch.tensor(x, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(r, t)      # values chosen exactly representable in fp32 or far from ties
    rng = np.random.default_rng(15)
    y = rng.normal(size=1000)
    assert np.all(np.abs(orc.round_to_bf16(y) - y) <= np.abs(y) * 2.0 ** -8)


def test_mask_guard_band_and_fp32_minmax_init_never_clips():
    """An element within 2^-10 of a quantization step outside a bound still counts
    as in range; with a min/max initialisation whose s was rounded to fp32 (so that
    the group maximum sits at Q_P(1 +- 2^-24)) nothing is clipped: db == 0 exactly,
    as Table 4 reports for the Asymm initialisation (E_clip = 0.0)."""
    spec = L4QSpec(rank=1, alpha=1.0, bits=2, group_size=4)          # unsigned grid [0, 3]
    s = np.array([[1.0]]); b = np.array([[0.0]])
    W0 = np.array([[-2.0 ** -12, 3.0 + 2.0 ** -12, -2.0 ** -9, 3.0 + 2.0 ** -9]])
    A = np.array([[1.0, 1.0, 1.0, 1.0]]); B = np.array([[0.0]])
    X = np.eye(4); dY = np.array([[1.0], [10.0], [100.0], [1000.0]])
    g = orc.backward(spec, X, dY, W0, A, B, s, b)
    assert g["dB"][0, 0] == 1.0 + 10.0                                # first two inside the guard band
    assert g["db"][0, 0] == 100.0 + 1000.0
    rng = np.random.default_rng(21)
    o, i, gsz = 16, 64, 16
    spec = L4QSpec(rank=2, alpha=4.0, bits=4, group_size=gsz)
    W0 = rng.normal(0, 0.02, (o, i)).astype(np.float32)
    Wg = W0.reshape(o, i // gsz, gsz)
    s32 = ((Wg.max(2) - Wg.min(2)) / np.float32(15)).astype(np.float32)
    b32 = Wg.min(2)
    A = rng.normal(size=(2, i)); B = np.zeros((o, 2))
    w = orc.prequant(spec, orc.merge(spec, W0, A, B), s32, b32)
    assert (w > 15).any()                                             # rounding of s does push some maxima past Q_P
    g = orc.backward(spec, rng.normal(size=(4, i)), rng.normal(size=(4, o)), W0, A, B, s32, b32)
    assert np.all(g["db"] == 0.0)


def test_guard_band_zero_is_the_printed_gate_and_changes_nothing_away_from_the_bounds():
    """App. A.1 prints the plain test Q_N <= w <= Q_P.  With mask_guard = 0 the oracle is that test: an element
    2^-12 of a step outside a bound is gated out.  And on a layer none of whose w lies within 2^-10 of a bound, the
    default band gives bit for bit the gradients of a scalar loop that applies the printed test element by element
    (Eq. 5-6 for ds, db; Eq. 13-14 for dA, dB), so the band only ever decides elements on a bound."""
    from dataclasses import replace
    spec0 = L4QSpec(rank=1, alpha=1.0, bits=2, group_size=4, mask_guard=0.0)
    s = np.array([[1.0]]); b = np.array([[0.0]])
    W0 = np.array([[-2.0 ** -12, 3.0 + 2.0 ** -12, 0.0, 3.0]])
    A = np.array([[1.0, 1.0, 1.0, 1.0]]); B = np.array([[0.0]])
    X = np.eye(4); dY = np.array([[1.0], [10.0], [100.0], [1000.0]])
    g = orc.backward(spec0, X, dY, W0, A, B, s, b)
    assert g["dB"][0, 0] == 100.0 + 1000.0                            # on the bounds: inside (inclusive)
    assert g["db"][0, 0] == 1.0 + 10.0                                # a hair outside: clipped

    rng = np.random.default_rng(33)
    spec, X, dY, W0, A, B, s, b = _layer(rng, o=5, i=24, r=3, M=7, g=8, bits=3, bscale=0.2, spread=0.8)
    qn, qp = orc.grid_bounds(spec)
    w = orc.prequant(spec, orc.merge(spec, W0, A, B), s, b)
    assert np.all(np.minimum(np.abs(w - qn), np.abs(w - qp)) > 2.0 ** -9)        # nobody near a bound ...
    assert (w < qn).any() and (w > qp).any() and ((w > qn) & (w < qp)).any()      # ... and all three branches occur
    got = orc.backward(spec, X, dY, W0, A, B, s, b)
    got0 = orc.backward(replace(spec, mask_guard=0.0), X, dY, W0, A, B, s, b)
    o, i = W0.shape
    gsz = spec.group_size
    G = dY.T @ X
    ds = np.zeros_like(s); db = np.zeros_like(b); Gm = np.zeros_like(G)
    for r_ in range(o):
        for c in range(i):
            k = c // gsz
            wv = w[r_, c]
            if wv < qn:
                ds[r_, k] += G[r_, c] * qn; db[r_, k] += G[r_, c]
            elif wv > qp:
                ds[r_, k] += G[r_, c] * qp; db[r_, k] += G[r_, c]
            else:
                ds[r_, k] += G[r_, c] * (np.rint(wv) - wv); Gm[r_, c] = G[r_, c]
    for res in (got, got0):
        np.testing.assert_allclose(res["ds"], ds, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(res["db"], db, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(res["dA"], spec.gamma * B.T @ Gm, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(res["dB"], spec.gamma * Gm @ A.T, rtol=1e-12, atol=1e-12)
    for k_ in ("dX", "dA", "dB", "ds", "db"):
        np.testing.assert_array_equal(got[k_], got0[k_])
