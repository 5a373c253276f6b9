"""Parity at the full sizes of the five workloads, in the launch configuration bench.py times
(tensor engine, symmetric tiles): sampled matrices against the oracle, properties for the rest."""
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


def _minimax_schedule(L=5):
    """The Polar-Express-style mapping: per-step quintics, each the minimax approximation of 1 on the image of the
    previous one, starting from [1e-3, 1] (the greedy construction that mapping is defined by; its authors' printed
    table is not available offline, so the coefficients are computed here), first step rescaled by 1.01 so that a
    rounded input slightly above 1 stays inside the interval. The first step's slope at the origin is 8.3."""
    from paper_2609_21102_b200 import schedules
    sched, _ = schedules.remez_sign_schedule(1e-3, L, margin=0.01)
    return [list(c) for c in sched]


def _check_samples(ctx, G, Om, k, p, J, sched, gamma, samples, tol, mode=0, band=(0.05, 1.6)):
    b, m, n = G.shape
    l = min(min(m, n), k + p)
    out, info = ctx.defl_polar_batched(G, k, p, J, sched, sketch=Om, gamma=gamma, restore_mode=mode,
                                       exploit_symmetry=True, want_info=True)
    torch.cuda.synchronize()
    assert int(info["status"].max()) == 0
    for i in samples:
        ref, s, kk, rho = oracle.deflated_polar(G[i].double().cpu().numpy(), k, l, Om[i].double().cpu().numpy(), J,
                                                oracle.schedule(sched), gamma=gamma, mode=mode)
        err = _rel(out[i].double().cpu().numpy(), ref)
        assert err <= tol, (i, err)
        assert abs(float(info["rho"][i]) - rho) <= 2e-3 * rho
        assert np.allclose(info["s"][i].double().cpu().numpy()[:k], s[:k], rtol=5e-3)
    # every matrix: finite, and its squared Frobenius norm is that of a matrix whose min(m,n) singular values
    # all lie in the band the quintic maps [0,1] into after a few steps (roughly [0.3, 1.25])
    o = out.float()
    assert bool(torch.isfinite(o).all())
    fro2 = (o * o).sum(dim=(1, 2)) / min(m, n)
    assert float(fro2.min()) > band[0] and float(fro2.max()) < band[1]
    return out


@pytest.mark.parametrize("shape_index,m,n", [(0, 768, 768), (1, 768, 3072)])
def test_workload2_gpt2_small_spiked(ctx, shape_index, m, n):
    dev = torch.device("cuda")
    G = inputs.workload_spiked(12, m, n, shape_index, device=dev).to(torch.bfloat16)
    Om = inputs.sketch(12, min(m, n), 16, 2, shape_index, device=dev)
    _check_samples(ctx, G, Om, 8, 8, 1, [MUON] * 5, 1.01, [0, 11], 3e-2)


@pytest.mark.parametrize("shape_index,n", [(0, 1024), (1, 3072), (2, 4096)])
def test_workload3_power_law_per_step_schedule(ctx, shape_index, n):
    dev = torch.device("cuda")
    G = inputs.workload_power_law(24, 1024, n, 3, shape_index, 0.8, 50.0, device=dev).to(torch.bfloat16)
    Om = inputs.sketch(24, 1024, 24, 3, shape_index, device=dev)
    _check_samples(ctx, G, Om, 16, 8, 1, _minimax_schedule(), 1.1, [23], 1e-2)


# Storage of the filter's iterates on workload 4 (error against the fp64 oracle, 1600 x 6400 group / square group):
# bf16 in every step 4.2e-2 / 2.8e-2; scaled IEEE half in the first step only 1.5e-2 / 1.1e-2; in the first two
# (the default) 1.07e-2 / 8.2e-3; in all five 5.5e-3 / 3.9e-3; the bf16 rounding of the exact result alone is 1.7e-3.
# The cause is the storage rounding of X_t alone: the bf16 figure is the same to four digits on the
# exact-fp32-product engine with A_t and B_t held in fp32, and it drops to 1e-5 with fp32 storage (measured).
# Rounding X_t (relative 2^-9 per entry in bf16) tilts each small singular direction by about
# 1e-3 * ||X_t||_F / (sqrt(m) sigma_i), large for this spectrum (sigma_i = 200/i, floor 3.6e-3 after deflation) and
# the 4:1 aspect while sigma_i is still small, i.e. in the first steps: later steps can afford bf16.
TOL_DEFAULT_XL = 1.5e-2              # two half steps, then bf16 (spec tolerance for the bf16 path: 3e-2)
TOL_HALF_ITERATES_XL = 1e-2
TOL_BF16_ITERATES_XL_WIDE = 5e-2


def test_workload4_gpt2_xl_both_groups(ctx):
    dev = torch.device("cuda")
    for shape_index, (m, n), samples, tol in ((1, (1600, 1600), [0, 47], TOL_DEFAULT_XL), (0, (1600, 6400), [5], TOL_DEFAULT_XL)):
        G = inputs.workload_power_law(48, m, n, 4, shape_index, 1.0, 200.0, 1e-4, device=dev).to(torch.bfloat16)
        Om = inputs.sketch(48, 1600, 48, 4, shape_index, device=dev)
        _check_samples(ctx, G, Om, 32, 16, 2, [MUON] * 5, 1.01, samples, tol)
        _check_samples(ctx, G, Om, 32, 16, 2, _minimax_schedule(), 1.1, samples[:1], tol, band=(0.6, 1.3))
        if n == 6400:
            # same matrices with fp32 storage on the exact engine (4 of them): the kernels themselves are exact
            out32 = ctx.defl_polar_batched(G[:4].float().contiguous(), 32, 16, 2, [MUON] * 5, sketch=Om[:4].contiguous(),
                                           gamma=1.01)
            ref, *_ = oracle.deflated_polar(G[2].double().cpu().numpy(), 32, 48, Om[2].double().cpu().numpy(), 2,
                                            oracle.schedule([MUON] * 5), gamma=1.01)
            assert _rel(out32[2].double().cpu().numpy(), ref) <= 2e-3
            outb = ctx.defl_polar_batched(G[:4].contiguous(), 32, 16, 2, [MUON] * 5, sketch=Om[:4].contiguous(), gamma=1.01,
                                          exploit_symmetry=True, bf16_iterates=1)
            eb = _rel(outb[2].double().cpu().numpy(), ref)
            assert 2e-2 < eb <= TOL_BF16_ITERATES_XL_WIDE, eb       # the option does switch the storage type
            outh = ctx.defl_polar_batched(G[:4].contiguous(), 32, 16, 2, [MUON] * 5, sketch=Om[:4].contiguous(), gamma=1.01,
                                          exploit_symmetry=True, bf16_iterates=2)
            eh = _rel(outh[2].double().cpu().numpy(), ref)
            assert eh <= TOL_HALF_ITERATES_XL, eh
        del G, Om
        torch.cuda.empty_cache()


def test_workload4_add_mode_and_tall_orientation(ctx):
    dev = torch.device("cuda")
    G = inputs.workload_power_law(4, 6400, 1600, 4, 0, 1.0, 200.0, 1e-4, device=dev).to(torch.bfloat16)
    Om = inputs.sketch(4, 1600, 48, 4, 0, device=dev)
    _check_samples(ctx, G, Om, 32, 16, 2, [MUON] * 5, 1.01, [3], TOL_DEFAULT_XL, mode=1)


def test_workload5_sdp_sequence(ctx):
    """Oracle parity at n = 1024 on a drifting sequence (warm-up, then deflated calls); at n = 4096, where one
    fp64 oracle projection costs 3 TFLOP, the deflated projection is checked against a brute-force fp64
    eigendecomposition (torch.linalg.eigh on the GPU) instead."""
    from paper_2609_21102_b200 import binding
    dev = torch.device("cuda")
    sched = [[1.875, -1.25, 0.375]] * 7
    for n, oracle_checked in ((1024, True), (4096, False)):
        K, k = 16, 8
        x, lam = inputs.sdp_first(n, heads=k, head_mag=1.0e3, device=dev)
        V = inputs.randn((n, K), inputs.seed_for(5, 0, inputs.PURPOSE_BASIS), dev).float()
        v0 = inputs.gaussian_vector(n, 5, inputs.PURPOSE_LANCZOS, device=dev)
        Vo = None
        if oracle_checked:
            q, r = np.linalg.qr(V.double().cpu().numpy())
            Vo = q * np.sign(np.diag(r))[None, :]
        for t in range(4):
            X = x.float()
            warm = t < 2
            P, info = ctx.defl_psd_project(X, k, V, sched, gamma=1.1, lanczos_start=v0, warmup=warm,
                                           exploit_symmetry=True, want_info=True)
            torch.cuda.synchronize()
            assert int(info["status"][0]) == 0
            assert torch.equal(P, P.T)
            if oracle_checked:
                Po, Vo, lam_o, ndef, th = oracle.psd_project(X.double().cpu().numpy(), Vo, k, oracle.schedule(sched),
                                                             gamma=1.1, warmup=warm, lanczos_v0=v0.double().cpu().numpy())
                assert _rel(P.double().cpu().numpy(), Po) <= (4e-3 if warm else 2e-3), (n, t)
                assert abs(float(info["theta"][0]) - th) <= 2e-3 * th
            x = inputs.sdp_next(x, t + 1)
        # last (deflated) projection against the exact projection
        w, v = torch.linalg.eigh(X.double())
        exact = (v * w.clamp(min=0)) @ v.T
        assert float((P.double() - exact).norm() / exact.norm()) <= 1e-3
        lg = info["lam"].double().abs()
        assert torch.allclose(lg[:k], torch.full((k,), 1.0e3, dtype=torch.float64, device=dev), rtol=1e-3)
        del x, X, P, exact, w, v
        torch.cuda.empty_cache()
