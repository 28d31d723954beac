"""Pins of the oracle's LoRA (Eq. 1-2) and QAT-LoRA (Sec. 3.1) layers against things other than
their own formulas: reverse-mode differentiation of Eq. 1 by torch.autograd, the column-vector form
of Eq. 1 written token by token, the L4Q oracle in the cases where the layers coincide, linearity,
and the fine-grid limit."""
import numpy as np
import pytest
import torch

from oracle import l4q_oracle as orc


def _case(seed=0, M=7, o=6, i=16, r=2, g=8, bits=4, outliers=False):
    rng = np.random.default_rng(seed)
    spec = orc.L4QSpec(rank=r, alpha=3.0, bits=bits, group_size=g)
    W0 = rng.normal(0, 0.02, (o, i))
    if outliers:
        W0[rng.random(W0.shape) < 0.1] *= 6.0
    A = rng.uniform(-0.25, 0.25, (r, i))
    B = rng.normal(0, 0.05, (o, r))
    X = rng.normal(size=(M, i))
    dY = rng.normal(size=(M, o))
    return spec, X, dY, W0, A, B


def test_lora_forward_token_by_token():
    spec, X, _, W0, A, B = _case()
    Y = orc.lora_forward(spec, X, W0, A, B)
    for t in range(X.shape[0]):                      # Eq. 1 on one column vector x
        x = X[t]
        y = np.zeros(W0.shape[0])
        xa = np.array([sum(A[k, j] * x[j] for j in range(x.size)) for k in range(spec.rank)])
        for oo in range(W0.shape[0]):
            y[oo] = sum(W0[oo, j] * x[j] for j in range(x.size)) + (spec.alpha / spec.rank) * sum(
                B[oo, k] * xa[k] for k in range(spec.rank))
        assert np.allclose(Y[t], y, rtol=1e-12, atol=1e-14)


def test_lora_backward_is_the_gradient_of_eq1():
    spec, X, dY, W0, A, B = _case(seed=1)
    tX, tA, tB = (torch.tensor(v, dtype=torch.float64, requires_grad=True) for v in (X, A, B))
    Y = tX @ torch.tensor(W0).T + spec.gamma * ((tX @ tA.T) @ tB.T)
    (Y * torch.tensor(dY)).sum().backward()
    g = orc.lora_backward(spec, X, dY, W0, A, B)
    assert np.allclose(g["dX"], tX.grad.numpy(), rtol=1e-12, atol=1e-14)
    assert np.allclose(g["dA"], tA.grad.numpy(), rtol=1e-12, atol=1e-14)
    assert np.allclose(g["dB"], tB.grad.numpy(), rtol=1e-12, atol=1e-14)


def test_lora_backward_finite_difference_in_one_entry():
    spec, X, dY, W0, A, B = _case(seed=2)
    g = orc.lora_backward(spec, X, dY, W0, A, B)
    loss = lambda A_, B_: float((orc.lora_forward(spec, X, W0, A_, B_) * dY).sum())
    h = 1e-6
    Ap = A.copy(); Ap[1, 5] += h
    Am = A.copy(); Am[1, 5] -= h
    assert (loss(Ap, B) - loss(Am, B)) / (2 * h) == pytest.approx(g["dA"][1, 5], rel=1e-7)
    Bp = B.copy(); Bp[3, 0] += h
    Bm = B.copy(); Bm[3, 0] -= h
    assert (loss(A, Bp) - loss(A, Bm)) / (2 * h) == pytest.approx(g["dB"][3, 0], rel=1e-7)


def _asymm(spec, W0):
    return orc.init_params(spec, W0, "asymm")


def test_qat_lora_with_zero_B_is_l4q_with_zero_B():
    spec, X, dY, W0, A, B = _case(seed=3, outliers=True)
    s, b = _asymm(spec, W0)
    s = s * 0.8                                       # shrink the range so that some weights clip
    Z = np.zeros_like(B)
    assert np.array_equal(orc.qat_lora_forward(spec, X, W0, A, Z, s, b), orc.forward(spec, X, W0, A, Z, s, b))
    gq = orc.qat_lora_backward(spec, X, dY, W0, A, Z, s, b)
    gl = orc.backward(spec, X, dY, W0, A, Z, s, b)
    for k in ("dX", "ds", "db"):
        assert np.allclose(gq[k], gl[k], rtol=1e-13, atol=1e-15), k
    assert np.abs(gl["db"]).max() > 0                 # the case does clip
    # dB differs exactly by the clipped part of G: L4Q gates G with the STE mask, LoRA does not
    assert not np.allclose(gq["dB"], gl["dB"])
    s2, b2 = _asymm(spec, W0)                         # nothing clips: every gate is open, dB coincides
    gq2 = orc.qat_lora_backward(spec, X, dY, W0, A, Z, s2, b2)
    gl2 = orc.backward(spec, X, dY, W0, A, Z, s2, b2)
    assert np.all(gl2["db"] == 0.0)
    assert np.allclose(gq2["dB"], gl2["dB"], rtol=1e-12, atol=1e-15)


def test_qat_lora_is_quantized_base_plus_lora_path():
    spec, X, dY, W0, A, B = _case(seed=4, outliers=True)
    s, b = _asymm(spec, W0)
    Z = np.zeros_like(B)
    Y = orc.qat_lora_forward(spec, X, W0, A, B, s, b)
    want = orc.forward(spec, X, W0, A, Z, s, b) + orc.lora_forward(spec, X, W0, A, B) - X @ W0.T
    assert np.allclose(Y, want, rtol=1e-12, atol=1e-14)
    g = orc.qat_lora_backward(spec, X, dY, W0, A, B, s, b)
    gl = orc.lora_backward(spec, X, dY, W0, A, B)
    g0 = orc.backward(spec, X, dY, W0, A, Z, s, b)
    assert np.allclose(g["dA"], gl["dA"], rtol=1e-13, atol=0) and np.allclose(g["dB"], gl["dB"], rtol=1e-13, atol=0)
    assert np.allclose(g["dX"], g0["dX"] + gl["dX"] - dY @ W0, rtol=1e-12, atol=1e-14)
    # the quantizer's gradients do not see the LoRA factors (Sec. 3.1, the decoupling of the two updates)
    assert np.array_equal(g["ds"], g0["ds"]) and np.array_equal(g["db"], g0["db"])
    # ... while L4Q's do
    assert not np.allclose(orc.backward(spec, X, dY, W0, A, B * 20, s, b)["ds"], g0["ds"])


def test_qat_lora_tends_to_lora_on_a_fine_grid():
    spec, X, dY, W0, A, B = _case(seed=5, bits=8)
    s, b = _asymm(spec, W0)
    Y = orc.qat_lora_forward(spec, X, W0, A, B, s, b)
    Yl = orc.lora_forward(spec, X, W0, A, B)
    bound = 0.5 * s.max() * np.abs(X).sum(axis=1).max()          # |W_q - W0| <= s/2 inside the range
    assert np.abs(Y - Yl).max() <= bound and np.abs(Y - Yl).max() > 0
    dX = orc.qat_lora_backward(spec, X, dY, W0, A, B, s, b)["dX"]
    dXl = orc.lora_backward(spec, X, dY, W0, A, B)["dX"]
    assert np.abs(dX - dXl).max() <= 0.5 * s.max() * np.abs(dY).sum(axis=1).max()


def test_planted_mistakes_are_caught():
    # a transposed factor or a dropped gamma in the LoRA gradient changes the autograd comparison
    spec, X, dY, W0, A, B = _case(seed=6)
    tA = torch.tensor(A, requires_grad=True)
    Y = torch.tensor(X) @ torch.tensor(W0).T + spec.gamma * ((torch.tensor(X) @ tA.T) @ torch.tensor(B).T)
    (Y * torch.tensor(dY)).sum().backward()
    wrong_no_gamma = (dY @ B).T @ X
    assert not np.allclose(wrong_no_gamma, tA.grad.numpy())
    assert np.allclose(spec.gamma * wrong_no_gamma, tA.grad.numpy())
