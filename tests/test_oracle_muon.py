"""Pins for the oracle's Deflated Muon step (Section 1, "Two applications": W <- W - lambda polar(M); Section 3,
"Muon with deflation"): expected values come from numpy/LAPACK SVDs, exact arithmetic identities and hand-worked
roundings, never from the oracle itself."""
import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(26092)


def _polar(M):
    u, s, vt = np.linalg.svd(M, full_matrices=False)
    return u @ vt


def _conditioned(m, n, lo=0.6, hi=1.8):
    """A matrix with singular values in [lo, hi]: the classical filter reaches its polar factor to rounding."""
    r = min(m, n)
    u, _ = np.linalg.qr(RNG.standard_normal((m, r)))
    v, _ = np.linalg.qr(RNG.standard_normal((n, r)))
    return (u * RNG.uniform(lo, hi, r)) @ v.T


def _headed(m, n):
    """Three leading singular values (3, 2.5, 2) over a bulk in [0.5, 1]: the gap 0.5 lets 25 subspace iterations
    find the leading triplets to rounding, so that deflation is exact and Eq. 3 applies."""
    r = min(m, n)
    u, _ = np.linalg.qr(RNG.standard_normal((m, r)))
    v, _ = np.linalg.qr(RNG.standard_normal((n, r)))
    s = np.concatenate([[3.0, 2.5, 2.0], RNG.uniform(0.5, 1.0, r - 3)])
    return (u * s) @ v.T


def test_round_to_storage_bf16_hand_worked_values():
    # bf16 keeps 8 significant bits: the spacing at 1.0 is 2^-7
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -(1.0 + 2.0 ** -8), 0.0, 3.0e38])
    want = np.array([1.0, 1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7, -1.0, 0.0, 2.0 ** 127 * (1 + 98 / 128)])   # 3.0e38 = 2^127 x 1.76324: 97.7 spacings -> 98
    got = oracle.round_to_storage(x, "bf16")
    assert np.array_equal(got, want)          # ties go to the even mantissa, sign symmetric
    assert np.array_equal(oracle.round_to_storage(x[:4], "f32"), x[:4].astype(np.float32).astype(np.float64))
    assert np.array_equal(oracle.round_to_storage(x[:4], None), x[:4])


def test_zero_learning_rate_leaves_weights_and_updates_momentum_exactly():
    m, n = 12, 20
    W, Mom, G = RNG.standard_normal((m, n)), RNG.standard_normal((m, n)), RNG.standard_normal((m, n))
    W1, M1 = oracle.muon_step(W, Mom, G, 0.0, 0.9, 0, 0, None, 0, [oracle.MUON_QUINTIC] * 5)
    assert np.array_equal(W1, W)
    assert np.allclose(M1, 0.9 * Mom + G, rtol=0, atol=1e-15)


@pytest.mark.parametrize("shape", [(24, 16), (16, 24)])
@pytest.mark.parametrize("nesterov", [False, True])
@pytest.mark.parametrize("k", [0, 3])
def test_step_is_w_minus_lr_polar_of_the_momentum(shape, nesterov, k):
    """With the classical quintic and enough steps the filter reaches polar(D) to rounding, so the step must equal
    the paper's W - lambda polar(M) computed from LAPACK's SVD (Section 1), for M = the updated momentum or its
    Nesterov look-ahead, with or without deflation (Eq. 3)."""
    m, n = shape
    lr, mu = 0.02, 0.95
    W = RNG.standard_normal((m, n))
    Mom = _headed(m, n)
    G = 1e-3 * RNG.standard_normal((m, n))          # small: the momentum keeps its gap
    Om = RNG.standard_normal((min(m, n), k + 3))
    M1 = mu * Mom + G
    D = G + mu * M1 if nesterov else M1
    want = W - lr * _polar(D)
    W1, Mret = oracle.muon_step(W, Mom, G, lr, mu, k, k + 3 if k else 0, Om, 25, [oracle.CLASSICAL_QUINTIC] * 30,
                                nesterov=nesterov, gamma=1.0, mode=oracle.PADDED)
    assert np.allclose(Mret, M1, rtol=0, atol=1e-15)
    assert np.linalg.norm(W1 - want) <= 1e-8 * np.linalg.norm(lr * _polar(D))


def test_weight_decay_and_scale_enter_linearly():
    m, n = 10, 14
    lr, wd = 0.1, 0.3
    W, Mom = RNG.standard_normal((m, n)), _conditioned(m, n)
    sched = [oracle.CLASSICAL_QUINTIC] * 30
    base, _ = oracle.muon_step(W, Mom, None, lr, 0.9, 0, 0, None, 0, sched)
    both, Mret = oracle.muon_step(W, Mom, None, lr, 0.9, 0, 0, None, 0, sched, weight_decay=wd, scale=2.5)
    assert np.array_equal(Mret, Mom)                      # no gradient: the momentum is taken as it is
    polar = _polar(Mom)
    assert np.allclose(base, W - lr * polar, atol=1e-10)
    assert np.allclose(both, (1 - lr * wd) * W - lr * 2.5 * polar, atol=1e-10)


def test_momentum_is_kept_in_the_storage_type():
    m, n = 8, 8
    W, Mom, G = np.zeros((m, n)), RNG.standard_normal((m, n)), RNG.standard_normal((m, n))
    _, M1 = oracle.muon_step(W, Mom, G, 0.0, 0.9, 0, 0, None, 0, [oracle.MUON_QUINTIC], storage="bf16")
    exact = 0.9 * Mom + G
    assert np.all(np.abs(M1 - exact) <= np.abs(exact) * 2.0 ** -8 + 1e-300)       # half a bf16 spacing
    assert np.array_equal(M1.astype(np.float32).view(np.uint32) & 0xFFFF, np.zeros((m, n), dtype=np.uint32))
