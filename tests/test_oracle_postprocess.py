"""Pins for the oracle's logit post-processing (App. B "Models": guidance,
temperature, top-k) against exact rational arithmetic, library routines and
identities."""
from fractions import Fraction

import numpy as np
import torch

import oracle


def _round_f32_exact(x: Fraction) -> float:
    """Round a rational to float32, round-half-even, with integer arithmetic only."""
    if x == 0:
        return 0.0
    sign = -1 if x < 0 else 1
    x = abs(x)
    e = 0
    while x >= 2:
        x /= 2
        e += 1
    while x < 1:
        x *= 2
        e -= 1
    assert e > -120          # normal range only in these tests
    scaled = x * (1 << 23)   # in [2^23, 2^24)
    n = scaled.numerator // scaled.denominator
    rem = scaled - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return sign * float(n) * 2.0 ** (e - 23)


def test_fma_single_rounding_adversarial():
    # (1+x)(1-x) + c with c = 2^24+2: the exact sum lies just below a float32
    # midpoint; rounding the double sum first would round the wrong way.
    for i in (1, 3, 77, 255):
        a = np.float32(1 + i * 2.0 ** -23)
        b = np.float32(1 - i * 2.0 ** -23)
        c = np.float32(2.0 ** 24 + 2)
        exact = Fraction(float(a)) * Fraction(float(b)) + Fraction(float(c))
        want = _round_f32_exact(exact)
        assert want == 2.0 ** 24 + 2
        got = float(oracle.fma_f32(a, b, c))
        assert got == want
        naive = float(np.float32(float(a) * float(b) + float(c)))
        assert naive != want      # the trap is real


def test_fma_matches_exact_rational_random():
    rng = np.random.default_rng(1)
    a = rng.standard_normal(400).astype(np.float32)
    b = (rng.standard_normal(400) * 3).astype(np.float32)
    c = (rng.standard_normal(400) * np.exp(rng.uniform(-12, 12, 400))).astype(np.float32)
    got = oracle.fma_f32(a, b, c)
    for i in range(400):
        exact = Fraction(float(a[i])) * Fraction(float(b[i])) + Fraction(float(c[i]))
        assert float(got[i]) == _round_f32_exact(exact)


def test_guidance_scale_one_is_cond_row():
    rng = np.random.default_rng(2)
    c = rng.standard_normal(64).astype(np.float32)
    u = rng.standard_normal(64).astype(np.float32)
    z = oracle.combine_f32(c, u, 1.0, 1.0)
    # 1*(c-u)+u: c up to the roundings of the difference and of the sum
    assert np.all(np.abs(z - c) <= np.spacing(np.abs(c)) + np.spacing(np.abs(c - u)))
    z0 = oracle.combine_f32(c, u, 0.0, 1.0)
    assert np.array_equal(z0, u)


def test_matches_torch_softmax_and_topk():
    g = torch.Generator().manual_seed(3)
    V = 512
    c = torch.randn(V, generator=g) * 2
    u = torch.randn(V, generator=g) * 2
    gsc, tau, k = 3.0, 0.7, 40
    P, z = oracle.postprocess_row(c.numpy(), u.numpy(), gsc, tau, k)
    zt = (u.double() + gsc * (c.double() - u.double())) / tau
    vals, idx = torch.topk(zt, k)
    ref = torch.zeros(V, dtype=torch.float64)
    ref[idx] = torch.softmax(vals, dim=0)
    assert np.count_nonzero(P) == k
    assert set(np.nonzero(P)[0]) == set(idx.tolist())
    assert np.allclose(P, ref.numpy(), atol=1e-6)
    assert abs(P.sum() - 1) < 1e-12
    # top_k >= V: plain softmax with temperature
    P2, _ = oracle.postprocess_row(c.numpy(), None, 1.0, tau, V)
    ref2 = torch.softmax(c.double() / tau, dim=0).numpy()
    assert np.allclose(P2, ref2, atol=1e-7)


def test_topk_keeps_ties_and_mask():
    row = np.array([1.0, 3.0, 2.0, 3.0, 2.0, 0.0, 2.0, -1.0], dtype=np.float32)
    P, z = oracle.postprocess_row(row, None, 1.0, 1.0, 3)
    # third largest is 2.0; all three entries equal to it are kept
    assert list(np.nonzero(P)[0]) == [1, 2, 3, 4, 6]
    e = np.exp(np.array([3, 2, 3, 2, 2.0]) - 3)
    assert np.allclose(P[[1, 2, 3, 4, 6]], e / e.sum(), atol=1e-15)
    P, z = oracle.postprocess_row(row, None, 1.0, 1.0, 0, allowed_begin=2, allowed_end=6)
    assert list(np.nonzero(P)[0]) == [2, 3, 4, 5]
    assert np.all(np.isneginf(z[[0, 1, 6, 7]]))
    # top-k counts only allowed entries
    P, _ = oracle.postprocess_row(row, None, 1.0, 1.0, 1, allowed_begin=4, allowed_end=8)
    assert list(np.nonzero(P)[0]) == [4, 6]
