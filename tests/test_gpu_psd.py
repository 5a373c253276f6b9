"""Parity of defl_psd_project with the fp64 CPU oracle (Algorithm 2), tolerance 2e-3 relative Frobenius on P (the bar of
the fp32/tf32 path), plus the bulk-only error (P minus its restored head), which the head would otherwise hide."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_21102_b200 import inputs

pytestmark = pytest.mark.gpu
TOL = 2e-3
# tf32 products on an input whose head has NOT been removed (warm-up calls, or the first call with a random
# basis) are the hardest case for the tensor path (rounding in the cross terms between head and bulk directions is
# multiplied by the head's magnitude in Z g(Z/theta), the effect deflation removes); they meet the same bound.
TOL_TF32_UNDEFLATED = 2e-3


@pytest.fixture(scope="module")
def ctx():
    from paper_2609_21102_b200 import binding
    c = binding.Context(0)
    yield c
    c.close()


def _rel(a, b):
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def _orth(V):
    q, r = np.linalg.qr(V)
    return q * np.sign(np.diag(r))[None, :]


def _sdp_like(n, heads, head_mag, seed):
    lam = torch.cat([head_mag * torch.where(inputs.rand((heads,), seed + 3) < 0.5, -1.0, 1.0).double(),
                     2.0 * inputs.rand((n - heads,), seed + 5) - 1.0])
    q = inputs.haar(n, n, seed)
    x = (q * lam.unsqueeze(0)) @ q.T
    return 0.5 * (x + x.T), lam, q


SCHED7 = [[1.875, -1.25, 0.375]] * 7


@pytest.mark.parametrize("n,K,k", [(256, 8, 4), (200, 6, 3), (384, 16, 8)])
@pytest.mark.parametrize("engine_name", ["tensor", "simt", "half"])
def test_psd_matches_oracle_with_tracked_basis(ctx, n, K, k, engine_name):
    """engine "half": the filter steps in IEEE half precision (the paper's SDP runs use the filter in half
    precision, Appendix E.2, "Composite Minimax Filter"), everything around them unchanged; same oracle, same tolerance."""
    from paper_2609_21102_b200 import binding
    engine = binding.ENGINE_SIMT if engine_name == "simt" else binding.ENGINE_AUTO
    half = engine_name == "half"
    X64, lam, q = _sdp_like(n, k, 50.0, 600 + n)
    X = X64.float().cuda()
    V0 = inputs.randn((n, K), 77 + n).float()
    v0 = inputs.gaussian_vector(n, 5, inputs.PURPOSE_LANCZOS).cuda()
    Vg = V0.clone().cuda()
    Vo = _orth(V0.double().numpy())
    Xo = X.double().cpu().numpy()
    for it in range(3):          # three block steps on a static matrix: the basis converges on both sides
        P, info = ctx.defl_psd_project(X, k, Vg, SCHED7, gamma=1.1, lanczos_start=v0, engine=engine, want_info=True,
                                       half_filter=half)
        torch.cuda.synchronize()
        Po, Vo_next, lam_o, ndef, theta_o = oracle.psd_project(Xo, Vo, k, oracle.schedule(SCHED7), gamma=1.1,
                                                               lanczos_v0=v0.double().cpu().numpy())
        assert int(info["status"][0]) == 0
        Pg = P.double().cpu().numpy()
        assert np.array_equal(Pg, Pg.T)
        tol = TOL_TF32_UNDEFLATED if (it == 0 and engine_name != "simt") else TOL
        assert _rel(Pg, Po) <= tol, (it, _rel(Pg, Po))
        assert abs(float(info["theta"][0]) - theta_o) <= 1e-3 * theta_o
        lg = info["lam"].double().cpu().numpy()
        assert np.allclose(np.sort(np.abs(lg[:k])), np.sort(np.abs(lam_o[:k])), rtol=1e-4)
        # the updated bases span the same space (unique QR factor up to rounding)
        Vn = Vg.double().cpu().numpy()
        assert np.allclose(Vn.T @ Vn, np.eye(K), atol=1e-4)
        assert np.linalg.norm(Vn - Vo_next @ (Vo_next.T @ Vn)) <= 5e-3 * np.sqrt(K)
        Vo = Vo_next
    # bulk-only error on the last projection: remove the positive head that both sides restore
    w, v = np.linalg.eigh(Xo)
    idx = np.argsort(-np.abs(w))[:k]
    head = (v[:, idx] * np.maximum(w[idx], 0)) @ v[:, idx].T
    bulk_err = np.linalg.norm((Pg - head) - (Po - head)) / np.linalg.norm(Po - head)
    assert bulk_err <= 2e-2, bulk_err


def test_psd_undeflated_baseline_and_frobenius_scale(ctx):
    from paper_2609_21102_b200 import binding
    n = 192
    X64, lam, q = _sdp_like(n, 2, 20.0, 901)
    X = X64.float().cuda()
    Xo = X.double().cpu().numpy()
    v0 = inputs.gaussian_vector(n, 5, inputs.PURPOSE_LANCZOS, 1).cuda()
    # k = 0, no basis: Eq. 7 with the Lanczos scale
    P, info = ctx.defl_psd_project(X, 0, None, SCHED7, lanczos_start=v0, want_info=True)
    Po, _, _, ndef, th = oracle.psd_project(Xo, None, 0, oracle.schedule(SCHED7), lanczos_v0=v0.double().cpu().numpy())
    assert ndef == 0
    assert abs(float(info["theta"][0]) - th) <= 1e-3 * th
    assert _rel(P.double().cpu().numpy(), Po) <= TOL_TF32_UNDEFLATED
    Pe = ctx.defl_psd_project(X, 0, None, SCHED7, lanczos_start=v0, engine=binding.ENGINE_SIMT)
    assert _rel(Pe.double().cpu().numpy(), Po) <= 1e-4          # exact fp32 products
    # warm-up flag with a basis: same projection, basis still advanced
    Vg = torch.from_numpy(_orth(inputs.randn((n, 4), 5).numpy())).float().cuda()
    Vin = Vg.double().cpu().numpy()
    P2 = ctx.defl_psd_project(X, 2, Vg, SCHED7, lanczos_start=v0, warmup=True)
    assert _rel(P2.double().cpu().numpy(), Po) <= TOL_TF32_UNDEFLATED
    _, Vn_o, *_ = oracle.psd_project(Xo, Vin, 2, oracle.schedule(SCHED7), warmup=True, lanczos_v0=v0.double().cpu().numpy())
    Vn = Vg.double().cpu().numpy()
    assert np.linalg.norm(Vn - Vn_o @ (Vn_o.T @ Vn)) <= 5e-3
    # Frobenius scale option
    P3, info3 = ctx.defl_psd_project(X, 0, None, SCHED7, norm_mode=binding.NORM_FROBENIUS, want_info=True)
    Po3, *_, th3 = oracle.psd_project(Xo, None, 0, oracle.schedule(SCHED7), norm_mode=oracle.NORM_FROBENIUS)
    assert abs(float(info3["theta"][0]) - th3) <= 1e-5 * th3
    assert _rel(P3.double().cpu().numpy(), Po3) <= TOL_TF32_UNDEFLATED


def test_psd_generated_start_vector_is_the_documented_generator(ctx):
    n = 128
    X64, *_ = _sdp_like(n, 2, 10.0, 31)
    X = X64.float().cuda()
    _, info = ctx.defl_psd_project(X, 0, None, SCHED7, seed=4242, want_info=True)
    v0 = oracle.fill_gaussian(n, 4242).astype(np.float32).astype(np.float64)
    th = oracle.lanczos_upper(X.double().cpu().numpy(), v0)
    assert abs(float(info["theta"][0]) - th) <= 1e-3 * th


def test_lanczos_breakdown_ends_the_krylov_space(ctx):
    """A start vector that is an eigenvector of R (exactly, in fp32): the recurrence breaks down after its first step,
    the Lanczos matrix is 1 x 1 (the rest zero padding, the later basis vectors never written) and the scale is the
    magnitude of that eigenvalue; a start vector inside a three-dimensional invariant subspace ends it after three."""
    n = 160
    d = np.concatenate([[2.0, -1.5, 1.25], 0.9 * (2.0 * inputs.rand((n - 3,), 88).double().numpy() - 1.0)])
    X = torch.diag(torch.tensor(d, dtype=torch.float32)).cuda()
    Xo = X.double().cpu().numpy()
    for support, want in (([0], 2.0), ([0, 1, 2], None)):
        v = np.zeros(n)
        v[support] = [1.0, 0.5, -0.25][:len(support)]
        v0 = torch.tensor(v, dtype=torch.float32).cuda()
        P, info = ctx.defl_psd_project(X, 0, None, SCHED7, lanczos_start=v0, want_info=True)
        th = oracle.lanczos_upper(Xo, v)
        Po, *_ = oracle.psd_project(Xo, None, 0, oracle.schedule(SCHED7), lanczos_v0=v)
        assert int(info["status"][0]) == 0
        assert abs(float(info["theta"][0]) - th) <= (1e-5 if want is not None else 1e-3) * th
        if want is not None:
            assert abs(th - want) <= 1e-12
        else:
            assert 2.0 * (1 - 1e-6) <= th <= 2.0 * (1 + 1e-3)        # the three Ritz values are the three eigenvalues
        assert _rel(P.double().cpu().numpy(), Po) <= TOL_TF32_UNDEFLATED


def test_psd_drifting_sequence_tracks_the_head(ctx):
    """A short synthetic stand-in for consecutive solver iterates: X_{t+1} = X_t + 1e-3 sym(N)."""
    n, K, k = 320, 16, 8
    X64, lam = inputs.sdp_first(n, heads=k, head_mag=1.0e3)
    V = inputs.randn((n, K), inputs.seed_for(5, 0, inputs.PURPOSE_BASIS)).float().cuda()
    Vo = _orth(V.double().cpu().numpy())
    v0 = inputs.gaussian_vector(n, 5, inputs.PURPOSE_LANCZOS).cuda()
    x = X64
    for t in range(4):
        X = x.float().cuda()
        warm = t < 2
        P, info = ctx.defl_psd_project(X, k, V, SCHED7, gamma=1.1, lanczos_start=v0, warmup=warm, want_info=True)
        Po, Vo, lam_o, ndef, th = oracle.psd_project(X.double().cpu().numpy(), Vo, k, oracle.schedule(SCHED7), gamma=1.1,
                                                     warmup=warm, lanczos_v0=v0.double().cpu().numpy())
        assert _rel(P.double().cpu().numpy(), Po) <= (TOL_TF32_UNDEFLATED if warm else TOL), t
        x = inputs.sdp_next(x, t + 1)
    lg = info["lam"].double().cpu().numpy()
    assert np.allclose(np.abs(lg[:k]), 1.0e3, rtol=1e-3)


def test_psd_argument_errors(ctx):
    from paper_2609_21102_b200 import binding
    X = torch.eye(64, device="cuda")
    V = torch.zeros((64, 4), device="cuda")
    with pytest.raises(binding.DeflError) as e:
        ctx.defl_psd_project(X, 5, V, SCHED7)              # k > K
    assert e.value.code == -2
    with pytest.raises(binding.DeflError) as e:
        ctx.defl_psd_project(X, 0, None, SCHED7, out=X)    # overlap
    assert e.value.code == -1


def test_psd_with_the_stage_one_minimax_schedule(ctx):
    """Appendix E.2, "Composite Minimax Filter"'s composite sign filter (stage one, eps = 1e-3, T = 7) as the schedule: parity with the oracle on
    the same schedule, and — because this filter reaches the sign function on [eps, 1] — closeness to the exact
    projection from LAPACK."""
    from paper_2609_21102_b200 import binding, schedules
    # (2 % margin: the minimax stages are only valid on [-1, 1] and the Lanczos scale is an estimate)
    sched, _ = schedules.remez_sign_schedule(1e-3, 7, margin=0.02)
    n, K, k = 384, 16, 8
    X64, lam, q = _sdp_like(n, k, 1.0e3, 4711)
    X = X64.float().cuda()
    Xo = X.double().cpu().numpy()
    v0 = inputs.gaussian_vector(n, 5, inputs.PURPOSE_LANCZOS, 2).cuda()
    # a basis that already holds the head to working accuracy (the state after the warm-up calls). A rough basis
    # will not do for this filter: with Ritz vectors off by 1e-3 the residual keeps eigenvalues of ~2 % of the
    # head (22 here), residual and padded directions overlap, X0 reaches eigenvalues of 1.5, and the minimax
    # stages, unlike the classical map, diverge outside [-1, 1]
    V = torch.from_numpy(_orth((q[:, :K] + 1e-7 * inputs.randn((n, K), 99)).numpy())).float().cuda()
    Vin = V.double().cpu().numpy()
    P = ctx.defl_psd_project(X, k, V, sched, gamma=1.1, lanczos_start=v0, exploit_symmetry=True)
    Po, *_ = oracle.psd_project(Xo, Vin, k, oracle.schedule(sched), gamma=1.1, lanczos_v0=v0.double().cpu().numpy())
    Pg = P.double().cpu().numpy()
    assert _rel(Pg, Po) <= TOL
    w, v = np.linalg.eigh(Xo)
    exact = (v * np.maximum(w, 0)) @ v.T
    idx = np.argsort(-np.abs(w))[:k]
    head = (v[:, idx] * np.maximum(w[idx], 0)) @ v[:, idx].T
    bulk = lambda M: np.linalg.norm((M - head) - (exact - head)) / np.linalg.norm(exact - head)
    assert bulk(Po) <= 1e-3          # the oracle with this filter is the projection up to eigenvalues below eps theta
    assert bulk(Pg) <= 2e-2          # tf32 against the exact projection, bulk only (measured 1.0e-2)


def test_half_filter_needs_the_tensor_engine_and_aligned_rows(ctx):
    from paper_2609_21102_b200 import binding
    X = torch.eye(200, device="cuda")
    with pytest.raises(binding.DeflError) as e:
        ctx.defl_psd_project(X, 0, None, SCHED7, engine=binding.ENGINE_SIMT, half_filter=True)
    assert e.value.code == -4
    with pytest.raises(binding.DeflError) as e:
        ctx.defl_psd_project(torch.eye(204, device="cuda"), 0, None, SCHED7, half_filter=True)     # 204 = 8 * 25.5
    assert e.value.code == -4
