"""The storage-sensitivity helpers used by the GPU parity tests: the roundings are the formats' roundings, and
the step-by-step evaluation, with no rounding, is the oracle's own whole-path result."""
import numpy as np
import pytest
import torch

import oracle
import storage_model as sm
from paper_2609_21102_b200 import inputs

MUON = list(oracle.MUON_QUINTIC)


def test_roundings_match_the_formats():
    rng = np.random.default_rng(5)
    x = rng.standard_normal(4096) * np.exp(rng.uniform(-6, 2, 4096))
    for name, unit, ref in (("half", 2.0 ** -11, None), ("bf16", 2.0 ** -8, torch.bfloat16), ("tf32", 2.0 ** -11, None)):
        r = sm.ROUNDERS[name](x)
        assert np.array_equal(sm.ROUNDERS[name](r), r)                       # idempotent
        normal = np.abs(x) * 32.0 >= 2.0 ** -14 if name == "half" else np.ones_like(x, dtype=bool)     # half: below that, gradual underflow
        assert float(np.max(np.abs(r - x)[normal] / np.abs(x)[normal])) <= unit * (1 + 1e-6)
        if ref is not None:
            assert np.array_equal(r, torch.tensor(x, dtype=torch.float32).to(ref).double().numpy())
    # half: values as torch's float16 keeps 32 x
    assert np.array_equal(sm.round_half_scaled(x), (torch.tensor(x * 32.0, dtype=torch.float64).to(torch.float16).double() / 32.0).numpy())
    # tf32 keeps 10 explicit mantissa bits: the low 13 bits of the fp32 pattern are zero
    bits = sm.round_tf32(x).astype(np.float32).view(np.uint32)
    assert int(np.bitwise_and(bits, 0x1FFF).max()) == 0


@pytest.mark.parametrize("m,n", [(96, 40), (40, 96)])
@pytest.mark.parametrize("add_mode", [False, True])
def test_stepwise_evaluation_is_the_oracle_path(m, n, add_mode):
    k, l, J, gamma, L = 4, 8, 1, 1.05, 4
    sigma = np.concatenate([[30.0, 20.0, 12.0, 8.0], np.linspace(1.0, 0.05, 36)])
    G = inputs.from_spectrum(m, n, sigma, 4242).numpy()
    Om = np.random.default_rng(3).standard_normal((min(m, n), l))
    ref, *_ = oracle.deflated_polar(G, k, l, Om, J, oracle.schedule([MUON] * L), gamma=gamma,
                                    mode=oracle.ADD if add_mode else oracle.PADDED)
    X0, head = sm.polar_entry(G, k, l, Om, J, gamma, add_mode)
    got = sm.filter_with_storage(X0, [MUON] * L, ["none"] * L) + (head if add_mode else 0.0)
    assert np.linalg.norm(got - ref) <= 1e-11 * np.linalg.norm(ref)
    got = sm.polar_filter_with_storage(X0, [MUON] * L, ["none"] * L) + (head if add_mode else 0.0)
    assert np.linalg.norm(got - ref) <= 1e-11 * np.linalg.norm(ref)
    assert sm.polar_storage_error(G, k, l, Om, J, [MUON] * L, gamma, add_mode, option=2) > 0.0
    # bf16 storage moves the result more than half storage does
    e_half = sm.polar_storage_error(G, k, l, Om, J, [MUON] * L, gamma, add_mode, option=2)
    e_bf16 = sm.polar_storage_error(G, k, l, Om, J, [MUON] * L, gamma, add_mode, option=1)
    assert e_bf16 > 2.0 * e_half


@pytest.mark.parametrize("warmup", [False, True])
def test_psd_pieces_rebuild_the_oracle_projection(warmup):
    n, K, k = 96, 8, 3
    lam = np.concatenate([[40.0, -30.0, 25.0], np.linspace(-1.0, 1.0, n - 3)])
    q = inputs.haar(n, n, 515).numpy()
    Z = (q * lam[None, :]) @ q.T
    Z = 0.5 * (Z + Z.T)
    Vb = np.linalg.qr(q[:, [0, 1, 2, 10, 20, 30, 40, 50]] + 1e-3 * inputs.randn((n, K), 516).numpy())[0]
    v0 = inputs.gaussian_vector(n, 5, inputs.PURPOSE_LANCZOS).double().numpy()
    sched = [list(oracle.CLASSICAL_QUINTIC)] * 7
    P, *_ = oracle.psd_project(Z, Vb, k, sched, gamma=1.1, warmup=warmup, lanczos_v0=v0)
    err, exact = sm.psd_storage_error(Z, Vb, k, sched, 1.1, warmup, v0, "tf32")
    assert np.linalg.norm(exact - P) <= 1e-10 * np.linalg.norm(P)
    assert 0.0 < err < 1e-2


def test_inv_root_storage_model_reduces_to_the_oracle_without_rounding():
    from oracle import inv_root
    rng = np.random.default_rng(5)
    n, k, p, T = 24, 2, 2, 5
    q, _ = np.linalg.qr(rng.standard_normal((n, n)))
    lam = np.concatenate([[400.0, 150.0], np.linspace(1.0, 0.1, n - 2)])
    A = (q * lam) @ q.T
    Vb = oracle.householder_orth(q[:, :3] + 1e-4 * rng.standard_normal((n, 3)))
    v0 = rng.standard_normal(n)
    err, exact = sm.inv_root_storage_error(A, Vb, k, p, T, 1.1, False, v0, fmt="none")
    want, *_ = inv_root.deflated_inv_root(A, Vb, k, p, T, gamma=1.1, lanczos_v0=v0)
    assert err <= 1e-13 and np.allclose(exact, want, atol=1e-12 * np.abs(want).max())
    err32, _ = sm.inv_root_storage_error(A, Vb, k, p, T, 1.1, False, v0, fmt="tf32")
    assert 1e-5 < err32 < 3e-3                      # 10 mantissa bits, a handful of stored matrices
