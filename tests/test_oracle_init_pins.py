"""Pins of the oracle's quantization-parameter initialisations (Sec. 3.3, Eq. 15; App. B) and
of the error sums of Table 4, against what the paper and arithmetic fix:
hand-computed values of a tiny group, the printed zero clipping of Asymm / L4Q_init at
initialisation (Table 4, "Initial" E_clip = 0.0), non-zero clipping of Symm / LSQ+ on data
built to overflow them, the signed <-> unsigned grid identity, and brute force."""
import numpy as np
import pytest

from oracle import l4q_oracle as orc


def _spec(bits=4, g=4, signed=True):
    return orc.L4QSpec(rank=1, alpha=1.0, bits=bits, group_size=g, signed_grid=signed)


def test_hand_computed_group():
    # one group {-0.8, 0.1, 0.3, 0.7}, 4 bits: Q_N = -8, Q_P = 7
    W = np.array([[-0.8, 0.1, 0.3, 0.7]])
    s, b = orc.init_params(_spec(), W, "l4q")
    assert s[0, 0] == pytest.approx(max(0.8 / 8, 0.7 / 7)) and b[0, 0] == 0.0           # Eq. 15
    s, b = orc.init_params(_spec(), W, "symm")
    assert s[0, 0] == pytest.approx(0.8 / 8) and b[0, 0] == 0.0
    s, b = orc.init_params(_spec(), W, "asymm")
    assert s[0, 0] == pytest.approx(1.5 / 15)
    assert b[0, 0] == pytest.approx(0.7 - 0.1 * 7) and b[0, 0] == pytest.approx(-0.8 + 0.1 * 8)
    mu, sigma = 0.075, np.sqrt(np.mean((W - 0.075) ** 2))
    s, b = orc.init_params(_spec(), W, "lsq+")
    assert s[0, 0] == pytest.approx(max(abs(mu - 3 * sigma), abs(mu + 3 * sigma)) / 8) and b[0, 0] == 0.0


def test_unsigned_grid_is_the_same_quantizer():
    rng = np.random.default_rng(0)
    W = rng.normal(0, 0.02, (6, 32))
    Z = (np.zeros((1, 32)), np.zeros((6, 1)))
    for m in orc.INIT_METHODS:
        ss, bs = orc.init_params(_spec(g=8, signed=True), W, m)
        su, bu = orc.init_params(_spec(g=8, signed=False), W, m)
        assert np.array_equal(ss, su) and np.allclose(bu, bs - 8 * ss, rtol=0, atol=1e-18)
        Wq_s = orc.fake_quant_weight(_spec(g=8, signed=True), W, *Z, ss, bs)[2]
        Wq_u = orc.fake_quant_weight(_spec(g=8, signed=False), W, *Z, su, bu)[2]
        assert np.allclose(Wq_s, Wq_u, rtol=0, atol=1e-15)
    # asymmetric initialisation on the unsigned grid is b = min, s = (max - min) / (2^n - 1)
    su, bu = orc.init_params(_spec(g=8, signed=False), W, "asymm")
    Wg = W.reshape(6, 4, 8)
    assert np.allclose(bu, Wg.min(2), atol=1e-17) and np.allclose(su, (Wg.max(2) - Wg.min(2)) / 15)


@pytest.mark.parametrize("signed", [True, False])
@pytest.mark.parametrize("bits", [3, 4])
def test_zero_clipping_at_initialisation_for_asymm_and_l4q(signed, bits):
    # Table 4, column "Initial": E_clip = 0.0 for Asymm and L4Q_init
    rng = np.random.default_rng(1)
    W = rng.normal(0, 0.02, (16, 256))
    W[rng.random(W.shape) < 0.01] *= 20.0                       # outliers
    spec = orc.L4QSpec(rank=2, alpha=4.0, bits=bits, group_size=64, signed_grid=signed)
    A, B = rng.normal(size=(2, 256)), np.zeros((16, 2))          # B = 0 at initialisation
    for m in ("asymm", "l4q"):
        s, b = orc.init_params(spec, W, m)
        e_quant, e_clip = orc.quant_error(spec, W, A, B, s, b)
        assert e_clip == 0.0 and e_quant > 0.0
        assert e_quant <= 0.5 * np.repeat(s, 64, axis=1).sum() * (1 + 1e-12)   # nothing clipped: |err| <= s/2


def test_symm_and_lsq_clip_what_they_cannot_represent():
    # Symm: the largest positive value maps to 2^(n-1) > Q_P; LSQ+: anything beyond 3 sigma overflows
    W = np.array([[0.8, -0.1, 0.2, 0.1]])
    spec = _spec()
    Z = (np.zeros((1, 4)), np.zeros((1, 1)))
    s, b = orc.init_params(spec, W, "symm")
    e_quant, e_clip = orc.quant_error(spec, W, *Z, s, b)
    assert e_clip == pytest.approx(0.8 - 7 * 0.1)                # clipped to Q_P * s
    W2 = np.array([[5.0] + [0.01 * (-1) ** k for k in range(31)]])
    spec2 = _spec(g=32)
    s, b = orc.init_params(spec2, W2, "lsq+")
    e_quant, e_clip = orc.quant_error(spec2, W2, np.zeros((1, 32)), np.zeros((1, 1)), s, b)
    assert e_clip == pytest.approx(5.0 - 7 * s[0, 0]) and e_clip <= e_quant


def test_quant_error_brute_force():
    rng = np.random.default_rng(2)
    spec = orc.L4QSpec(rank=2, alpha=3.0, bits=3, group_size=4, signed_grid=False)
    W0, A, B = rng.normal(0, 1, (3, 8)), rng.normal(0, 1, (2, 8)), rng.normal(0, 0.3, (3, 2))
    s, b = rng.uniform(0.2, 0.5, (3, 2)), rng.normal(-1.0, 0.2, (3, 2))
    eq = ec = 0.0
    for o in range(3):
        for j in range(8):
            wc = W0[o, j] + 1.5 * sum(B[o, k] * A[k, j] for k in range(2))
            w = (wc - b[o, j // 4]) / s[o, j // 4]
            wq = round(min(max(w, 0.0), 7.0)) * s[o, j // 4] + b[o, j // 4]
            eq += abs(wc - wq)
            if w < 0.0 - 2.0 ** -10 or w > 7.0 + 2.0 ** -10:
                ec += abs(wc - wq)
    got = orc.quant_error(spec, W0, A, B, s, b)
    assert got[0] == pytest.approx(eq, rel=1e-12) and got[1] == pytest.approx(ec, rel=1e-12) and ec > 0


def test_constant_group_gets_the_floor():
    s, b = orc.init_params(_spec(), np.zeros((1, 4)), "l4q")
    assert s[0, 0] == orc.S_FLOOR


# ---- fully quantized inference (Sec. 3.2, App. F) ----

def test_infer_equals_forward_when_the_export_is_lossless():
    # s and b + s Q_N exactly representable in fp16 => the export loses nothing and inference reproduces Eq. 10
    rng = np.random.default_rng(3)
    for bits, signed in ((4, False), (3, True)):
        spec = orc.L4QSpec(rank=2, alpha=4.0, bits=bits, group_size=32, signed_grid=signed)
        W0, A, B = rng.normal(0, 0.3, (5, 64)), rng.normal(0, 1, (2, 64)), rng.normal(0, 0.05, (5, 2))
        s = rng.integers(1, 8, (5, 2)) / 64.0                    # multiples of 2^-6: exact in fp16
        b = rng.integers(-32, 32, (5, 2)) / 32.0
        X = rng.normal(0, 1, (7, 64))
        codes, s16, b16 = orc.pack_int(spec, W0, A, B, s, b)
        assert np.array_equal(s16.astype(np.float64), s)
        Y = orc.forward(spec, X, W0, A, B, s, b)
        assert np.allclose(orc.infer(spec, X, codes, s16, b16), Y, rtol=1e-13, atol=1e-13)


def test_infer_brute_force_from_the_bitstream():
    rng = np.random.default_rng(4)
    spec = orc.L4QSpec(rank=1, alpha=1.0, bits=3, group_size=32)
    u = rng.integers(0, 8, (2, 32))
    words = np.zeros((2, 3), dtype=np.uint64)
    for o in range(2):
        for j in range(32):
            for k in range(3):                                   # bit k of code j sits at stream bit 3 j + k
                pos = 3 * j + k
                words[o, pos // 32] |= np.uint64(((int(u[o, j]) >> k) & 1) << (pos % 32))
    s16 = np.array([[0.25], [0.5]], dtype=np.float16)
    b16 = np.array([[-1.0], [0.125]], dtype=np.float16)
    X = rng.normal(0, 1, (3, 32))
    Y = [[sum(X[t, j] * (u[o, j] * float(s16[o, 0]) + float(b16[o, 0])) for j in range(32)) for o in range(2)]
         for t in range(3)]
    assert np.allclose(orc.infer(spec, X, words.astype(np.uint32), s16, b16), np.array(Y), rtol=1e-13)


# ---- AdamW (App. D) ----

def test_adamw_matches_the_library_optimizer():
    import torch
    rng = np.random.default_rng(5)
    p0 = rng.normal(0, 1, (7, 5))
    p_t = torch.tensor(p0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.AdamW([p_t], lr=3e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    p, m, v = p0.copy(), np.zeros_like(p0), np.zeros_like(p0)
    for step in range(1, 6):
        g = rng.normal(0, 1, p0.shape)
        p_t.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        p, m, v = orc.adamw_step(p, g, m, v, step, lr=3e-3)
        assert np.allclose(p, p_t.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_adamw_first_step_is_a_sign_step():
    # t = 1: mh = g, vh = g^2, so the update is -lr * g / (|g| + eps) on top of the decay
    p, g = np.array([1.0, -2.0, 0.5]), np.array([0.3, -4.0, 1e-3])
    got, _, _ = orc.adamw_step(p, g, np.zeros(3), np.zeros(3), 1, lr=0.1, weight_decay=0.0)
    assert np.allclose(got, p - 0.1 * g / (np.abs(g) + 1e-8), rtol=1e-12)
