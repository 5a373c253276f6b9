"""Numerical events are reported per matrix in defl_info.status and never end in a trap or a hang. Every failure here
is made on the host side (inputs, an environment override read at context creation): no kernel faults."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_21102_b200 import inputs

pytestmark = pytest.mark.gpu
MUON = [3.4445, -4.7750, 2.0315]


@pytest.fixture(scope="module")
def ctx():
    from paper_2609_21102_b200 import binding
    c = binding.Context(0)
    yield c
    c.close()


def _rel(a, b):
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def _gapped(b, m, n, k, dtype, seed):
    ms = min(m, n)
    sigma = np.concatenate([np.linspace(60.0, 30.0, k), np.linspace(1.0, 0.1, ms - k)])
    return torch.stack([inputs.from_spectrum(m, n, sigma, seed + i) for i in range(b)]).to(dtype)


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 2e-3), (torch.bfloat16, 3e-2)])
def test_cholesky_breakdown_takes_the_shifted_retry(ctx, dtype, tol):
    """A sketch with a zero column makes the panel's Gram matrix exactly singular: the Cholesky factorisation meets a
    zero pivot, restarts with a diagonal shift and says so. The lost direction is one of the oversampling ones; with a
    clear gap behind the k deflated values the result stays within the bar of the oracle (whose Householder step
    completes the basis with a direction of its own choice)."""
    from paper_2609_21102_b200 import binding
    b, m, n, k, p, J = 3, 160, 288, 4, 6, 1
    G = _gapped(b, m, n, k, dtype, 8100).cuda()
    Om = inputs.sketch(b, m, k + p, 1, 3).clone()
    Om[:, :, k + p - 1] = 0.0
    Om[1, :, k + 1] = 0.0
    Om = Om.cuda()
    out, info = ctx.defl_polar_batched(G, k, p, J, [MUON] * 5, sketch=Om, gamma=1.01, want_info=True)
    torch.cuda.synchronize()
    st = info["status"].cpu().tolist()
    assert all(s & binding.ST_CHOL_SHIFT for s in st), st
    assert all((s & ~binding.ST_CHOL_SHIFT) == 0 for s in st), st
    for i in range(b):
        ref, *_ = oracle.deflated_polar(G[i].double().cpu().numpy(), k, k + p, Om[i].double().cpu().numpy(), J,
                                        oracle.schedule([MUON] * 5), gamma=1.01)
        assert _rel(out[i].double().cpu().numpy(), ref) <= tol, i


def test_rank_deficient_input_stays_finite_and_close(ctx):
    """Rank 6 with a sketch of 8 columns: two sketch directions carry nothing but rounding noise. Whatever the
    factorisation makes of them (a shifted retry or a tiny pivot), the three deflated triplets and the result agree
    with the oracle, and no other event is raised."""
    from paper_2609_21102_b200 import binding
    b, m, n, k, p, J = 2, 96, 160, 3, 5, 1
    sigma = np.concatenate([[40.0, 25.0, 15.0, 1.0, 0.6, 0.3], np.zeros(90)])
    G = torch.stack([inputs.from_spectrum(m, n, sigma, 8200 + i) for i in range(b)]).float().cuda()
    Om = inputs.sketch(b, m, k + p, 1, 4).cuda()
    out, info = ctx.defl_polar_batched(G, k, p, J, [MUON] * 5, sketch=Om, gamma=1.01, want_info=True)
    torch.cuda.synchronize()
    assert all((s & ~binding.ST_CHOL_SHIFT) == 0 for s in info["status"].cpu().tolist())
    assert bool(torch.isfinite(out).all())
    for i in range(b):
        ref, s, *_ = oracle.deflated_polar(G[i].double().cpu().numpy(), k, k + p, Om[i].double().cpu().numpy(), J,
                                           oracle.schedule([MUON] * 5), gamma=1.01)
        assert np.allclose(info["s"][i, :k].double().cpu().numpy(), s[:k], rtol=1e-3)
        assert _rel(out[i].double().cpu().numpy(), ref) <= 2e-3, i


def test_jacobi_sweep_cap_is_reported(monkeypatch):
    """One sweep is never enough for a 12 x 12 core: the eigensolver stops at the cap and raises its bit."""
    from paper_2609_21102_b200 import binding
    monkeypatch.setenv("DEFL_JACOBI_SWEEPS", "1")
    c = binding.Context(0)
    G = _gapped(2, 128, 192, 6, torch.float32, 8300).cuda()
    out, info = c.defl_polar_batched(G, 6, 6, 1, [MUON] * 3, seed=5, want_info=True)
    torch.cuda.synchronize()
    assert all(s & binding.ST_JACOBI_CAP for s in info["status"].cpu().tolist())
    assert bool(torch.isfinite(out).all())
    c.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("k", [0, 4])
def test_non_finite_input_is_flagged_and_stays_in_its_matrix(ctx, dtype, k):
    """A NaN in one matrix of a batch: that matrix comes back non-finite and flagged (zero residual: its norm is
    not a number; non-finite result), its neighbours come back exactly as they do without it."""
    from paper_2609_21102_b200 import binding
    b, m, n, p = 3, 136, 200, 4
    G = _gapped(b, m, n, max(k, 1), dtype, 8400).cuda()
    Om = inputs.sketch(b, m, max(k + p, 1), 1, 5).cuda() if k else None
    clean, info0 = ctx.defl_polar_batched(G, k, p if k else 0, 1, [MUON] * 4, sketch=Om, gamma=1.01, want_info=True)
    assert info0["status"].cpu().tolist() == [0, 0, 0]
    Gn = G.clone()
    Gn[1, 7, 11] = float("nan")
    out, info = ctx.defl_polar_batched(Gn, k, p if k else 0, 1, [MUON] * 4, sketch=Om, gamma=1.01, want_info=True)
    torch.cuda.synchronize()
    st = info["status"].cpu().tolist()
    assert st[0] == 0 and st[2] == 0
    assert st[1] & binding.ST_ZERO_RESIDUAL and st[1] & binding.ST_NONFINITE
    assert not bool(torch.isfinite(out[1].float()).any())
    assert torch.equal(out[0], clean[0]) and torch.equal(out[2], clean[2])


def test_half_iterate_overflow_is_reported(ctx):
    """A schedule that diverges (a = 60 per step) drives the scaled IEEE half iterates of the bf16 path out of
    range: the result is not finite and the call says so, per matrix, instead of returning Inf with status 0."""
    from paper_2609_21102_b200 import binding
    G = _gapped(2, 128, 256, 2, torch.bfloat16, 8500).cuda()
    out, info = ctx.defl_polar_batched(G, 0, 0, 0, [[60.0, 0.0, 0.0]] * 6, want_info=True, bf16_iterates=2)
    torch.cuda.synchronize()
    assert all(s & binding.ST_NONFINITE for s in info["status"].cpu().tolist())
    fine, info2 = ctx.defl_polar_batched(G, 0, 0, 0, [MUON] * 5, want_info=True, bf16_iterates=2)
    assert info2["status"].cpu().tolist() == [0, 0] and bool(torch.isfinite(fine.float()).all())
