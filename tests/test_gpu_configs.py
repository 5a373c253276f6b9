"""Parity at the full sizes of the five workloads, in the launch configuration bench.py times
(tensor engine, symmetric tiles): sampled matrices against the oracle, properties for the rest."""
import numpy as np
import pytest
import torch

import oracle
import storage_model
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


def _scalar_band(sched, x_lo, x_hi, grid=4001):
    """Image of [x_lo, x_hi] under the composite scalar map p_L o ... o p_1, p_t(x) = a x + b x^3 + c x^5."""
    x = np.linspace(x_lo, x_hi, grid)
    for a, b, c in sched:
        x = a * x + b * x ** 3 + c * x ** 5
    return float(x.min()), float(x.max())


def _check_every_matrix(out, G, rho, sched, gamma, sigma_floor, slack):
    """Properties that hold for every matrix of the batch at any size, evaluated on the device in fp32/fp64:
    (1) out and G share their singular vectors (the filter acts on singular values only), so out G^T (short side) is
        symmetric positive semidefinite: a result that belongs to another matrix, or a transposed or permuted one, fails;
    (2) every singular value of out lies in the image of [sigma_floor / rho, 1] under the scalar composite map (after
        Frobenius normalisation the residual's singular values are at most 1, and the padded head sits at 1 / gamma)."""
    b, m, n = G.shape
    o, g = out.float(), G.float()
    S = o @ g.transpose(1, 2) if m <= n else o.transpose(1, 2) @ g
    skew = (S - S.transpose(1, 2)).flatten(1).norm(dim=1) / S.flatten(1).norm(dim=1)
    # (a result that belongs to another matrix gives a ratio near sqrt(2); storage rounding of the iterates leaves
    # 1e-2 to 5e-2, most with the steep first step of the per-step minimax schedule)
    assert float(skew.max()) <= 0.1, ("out G^T not symmetric", float(skew.max()))
    ev = torch.linalg.eigvalsh(0.5 * (S + S.transpose(1, 2)).double())
    assert float((ev.min(dim=1).values / ev.max(dim=1).values).min()) >= -slack, "out G^T not positive semidefinite"
    gram = (o @ o.transpose(1, 2) if m <= n else o.transpose(1, 2) @ o).double()
    sv = torch.linalg.eigvalsh(gram).clamp(min=0).sqrt()
    for i in range(b):
        lo, hi = _scalar_band(sched, sigma_floor / float(rho[i]), 1.0)
        assert float(sv[i].min()) >= lo - slack and float(sv[i].max()) <= hi + slack, (i, float(sv[i].min()), float(sv[i].max()), lo, hi)


def _check_samples(ctx, G, Om, k, p, J, sched, gamma, samples, tol, mode=0, sigma_floor=0.0, slack=6e-2):
    b, m, n = G.shape
    l = min(min(m, n), k + p)
    out, info = ctx.defl_polar_batched(G, k, p, J, sched, sketch=Om, gamma=gamma, restore_mode=mode,
                                       exploit_symmetry=True, want_info=True)
    torch.cuda.synchronize()
    assert int(info["status"].max()) == 0
    worst = 0.0
    for i in samples:
        ref, s, kk, rho = oracle.deflated_polar(G[i].double().cpu().numpy(), k, l, Om[i].double().cpu().numpy(), J,
                                                oracle.schedule(sched), gamma=gamma, mode=mode)
        err = _rel(out[i].double().cpu().numpy(), ref)
        worst = max(worst, err)
        assert err <= tol, (i, err)
        assert abs(float(info["rho"][i]) - rho) <= 2e-3 * rho
        assert np.allclose(info["s"][i].double().cpu().numpy()[:k], s[:k], rtol=5e-3)
    if G.dtype == torch.bfloat16 and samples:
        # the error is what the 16-bit storage of the filter's iterates, Gram matrices and polynomials (and of the bf16
        # result) explains for this input, measured on the oracle's side (the two agree to a few percent in norm; the
        # individual roundings differ, so the results themselves do not coincide): the kernels add nothing on top
        i = samples[0]
        model = storage_model.polar_storage_error(G[i].double().cpu().numpy(), k, l, Om[i].double().cpu().numpy(), J, sched,
                                                  gamma, mode == 1, round_output=True)
        e0 = _rel(out[i].double().cpu().numpy(), oracle.deflated_polar(G[i].double().cpu().numpy(), k, l, Om[i].double().cpu().numpy(), J,
                                                                       oracle.schedule(sched), gamma=gamma, mode=mode)[0])
        print("storage model for sample %d: %.3e (measured %.3e)" % (i, model, e0))
        assert e0 <= 1.5 * model + 1e-3, (i, e0, model)
    print("parity %dx%dx%d k=%d mode=%d samples=%s worst=%.3e (tol %.1e)" % (b, m, n, k, mode, samples, worst, tol))
    assert bool(torch.isfinite(out.float()).all())
    if mode == 0:
        _check_every_matrix(out, G, info["rho"].cpu(), sched, gamma, sigma_floor, slack)
    return out, worst


@pytest.mark.parametrize("shape_index,m,n", [(0, 768, 768), (1, 768, 3072)])
def test_workload2_gpt2_small_spiked(ctx, shape_index, m, n):
    dev = torch.device("cuda")
    G = inputs.workload_spiked(12, m, n, shape_index, device=dev).to(torch.bfloat16)
    Om = inputs.sketch(12, min(m, n), 16, 2, shape_index, device=dev)
    _check_samples(ctx, G, Om, 8, 8, 1, [MUON] * 5, 1.01, [0, 3, 7, 11], 3e-2)


@pytest.mark.parametrize("shape_index,n", [(0, 1024), (1, 3072), (2, 4096)])
def test_workload3_power_law_per_step_schedule(ctx, shape_index, n):
    dev = torch.device("cuda")
    G = inputs.workload_power_law(24, 1024, n, 3, shape_index, 0.8, 50.0, device=dev).to(torch.bfloat16)
    Om = inputs.sketch(24, 1024, 24, 3, shape_index, device=dev)
    _check_samples(ctx, G, Om, 16, 8, 1, _minimax_schedule(), 1.1, [0, 8, 16, 23], 1e-2, sigma_floor=50.0 * 1024 ** -0.8)


# Storage of the filter's iterates on workload 4 (error against the fp64 oracle, 1600 x 6400 group / square group):
# bf16 in every step 4.2e-2 / 2.8e-2; scaled IEEE half in the first step only 1.5e-2 / 1.1e-2; in the first two
# (the default) 1.07e-2 / 8.2e-3; in all five 5.5e-3 / 3.9e-3; the bf16 rounding of the exact result alone is 1.7e-3.
# The cause is the storage rounding of X_t alone: the bf16 figure is the same to four digits on the
# exact-fp32-product engine with A_t and B_t held in fp32, and it drops to 1e-5 with fp32 storage (measured).
# Rounding X_t (relative 2^-9 per entry in bf16) tilts each small singular direction by about
# 1e-3 * ||X_t||_F / (sqrt(m) sigma_i), large for this spectrum (sigma_i = 200/i, floor 3.6e-3 after deflation) and
# the 4:1 aspect while sigma_i is still small, i.e. in the first steps: later steps can afford bf16.
TOL_DEFAULT_XL = 1.5e-2              # two half steps, then bf16 (the bf16 path's bar is 3e-2)
TOL_HALF_ITERATES_XL = 1e-2
TOL_BF16_ITERATES_XL_WIDE = 5e-2
# SDP workload, deflated calls: error of P against the oracle relative to the bulk of P alone (tf32 filter)
TOL_SDP_BULK = 2e-3


def test_workload4_gpt2_xl_both_groups(ctx):
    dev = torch.device("cuda")
    for shape_index, (m, n), samples, tol in ((1, (1600, 1600), [0, 15, 31, 47], TOL_DEFAULT_XL), (0, (1600, 6400), [5, 17, 29, 41], TOL_DEFAULT_XL)):
        G = inputs.workload_power_law(48, m, n, 4, shape_index, 1.0, 200.0, 1e-4, device=dev).to(torch.bfloat16)
        Om = inputs.sketch(48, 1600, 48, 4, shape_index, device=dev)
        _check_samples(ctx, G, Om, 32, 16, 2, [MUON] * 5, 1.01, samples, tol, sigma_floor=0.125)
        _check_samples(ctx, G, Om, 32, 16, 2, _minimax_schedule(), 1.1, samples[:2], tol, sigma_floor=0.125)
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


def _bulk_norm(P, lam, n_deflated):
    """Frobenius norm of P without its restored positive head: the head's eigenvalues (about 1e3) carry almost all of
    ||P||_F (about 2e3 against 26 for the bulk), so an error is also judged against the bulk alone. The restored part
    is sum lambda_i u_i u_i^T over the deflated Ritz pairs with lambda_i > 0, orthogonal to the rest up to the
    Ritz residual: ||bulk||_F^2 = ||P||_F^2 - sum lambda_i^2."""
    head2 = float(sum(l * l for l in lam[:n_deflated] if l > 0))
    return float(np.sqrt(max(np.linalg.norm(P) ** 2 - head2, 0.0)))


def test_workload5_sdp_sequence(ctx):
    """The drifting SDP sequence (two warm-up calls, then deflated calls) against the oracle: every call at n = 1024;
    at n = 4096, where one fp64 oracle projection costs 3 TFLOP, the first deflated call (both sides start it from
    the same basis, the one the library produced during its warm-up calls). The error is judged on P as a whole and
    on the bulk alone; the last projection is also compared with an fp64 eigendecomposition."""
    dev = torch.device("cuda")
    sched = [[1.875, -1.25, 0.375]] * 7
    for n, oracle_calls in ((1024, (0, 1, 2, 3)), (4096, (2,))):
        K, k = 16, 8
        x, lam = inputs.sdp_first(n, heads=k, head_mag=1.0e3, device=dev)
        V = inputs.randn((n, K), inputs.seed_for(5, 0, inputs.PURPOSE_BASIS), dev).float()
        v0 = inputs.gaussian_vector(n, 5, inputs.PURPOSE_LANCZOS, device=dev)
        for t in range(4):
            X = x.float()
            warm = t < 2
            V_in = V.double().cpu().numpy()
            if t == 0:      # the library orthonormalises the Gaussian start block itself; the oracle wants it done
                q, r = np.linalg.qr(V_in)
                V_in = q * np.sign(np.diag(r))[None, :]
            P, info = ctx.defl_psd_project(X, k, V, sched, gamma=1.1, lanczos_start=v0, warmup=warm,
                                           exploit_symmetry=True, want_info=True)
            torch.cuda.synchronize()
            assert int(info["status"][0]) == 0
            assert torch.equal(P, P.T)
            if t in oracle_calls:
                Po, Vo, lam_o, ndef, th = oracle.psd_project(X.double().cpu().numpy(), V_in, k, oracle.schedule(sched),
                                                             gamma=1.1, warmup=warm, lanczos_v0=v0.double().cpu().numpy())
                Pg = P.double().cpu().numpy()
                assert _rel(Pg, Po) <= 2e-3, (n, t, _rel(Pg, Po))
                assert abs(float(info["theta"][0]) - th) <= 2e-3 * th
                if not warm:
                    assert ndef == k and int(info["k_used"][0]) == k
                    bulk = _bulk_norm(Po, lam_o, ndef)
                    assert 0.2 * np.sqrt(n) < bulk < np.sqrt(n)        # ||max(U(-1,1), 0)||_F is about sqrt(n / 6)
                    err_bulk = float(np.linalg.norm(Pg - Po)) / bulk
                    print("sdp n=%d call %d: whole %.3e bulk-only %.3e (bulk norm %.1f)" % (n, t, _rel(Pg, Po), err_bulk, bulk))
                    assert err_bulk <= TOL_SDP_BULK, (n, t, err_bulk)
                    # the updated bases span the same subspace
                    Vg = V.double().cpu().numpy()
                    assert _rel(Vg @ Vg.T, Vo @ Vo.T) <= 1e-3
                del Po, Pg
            x = inputs.sdp_next(x, t + 1)
        # last (deflated) projection against the exact projection
        w, v = torch.linalg.eigh(X.double())
        exact = (v * w.clamp(min=0)) @ v.T
        assert float((P.double() - exact).norm() / exact.norm()) <= 1e-3
        lg = info["lam"].double().abs()
        assert torch.allclose(lg[:k], torch.full((k,), 1.0e3, dtype=torch.float64, device=dev), rtol=1e-3)
        del x, X, P, exact, w, v
        torch.cuda.empty_cache()
