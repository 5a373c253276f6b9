"""defl_admm_diag_sdp on the GPU against the fp64 oracle loop (Appendix E.1, "ADMM for Standard-Form SDP"), iteration by iteration."""
import numpy as np
import pytest
import torch

import oracle
import storage_model
from paper_2609_21102_b200 import inputs

pytestmark = pytest.mark.gpu

SCHED = [list(oracle.CLASSICAL_QUINTIC)] * 10
# Per-iteration tolerance on S relative to ||S||_F: the library's bars (fp32 engine: rounding only; tf32 tensor engine
# and half filter: 2e-3). On the tensor engine the error is, besides, held to what the 11-bit storage of the filter's
# iterate, of its square and of the step's polynomial explains for that iteration's input, measured on the oracle's
# side (storage_model.psd_storage_error), times two: a kernel that adds an error of its own (an iterate that is not
# exactly symmetric, say, which the filter doubles at every step) fails this long before it reaches the bar.
TOL_ENGINE = {"fp32": 1e-4, "tf32": 2e-3, "half": 2e-3}      # "half": the filter steps in IEEE half
STORAGE = {"tf32": "tf32", "half": "half1"}


@pytest.fixture(scope="module")
def ctx():
    from paper_2609_21102_b200 import binding
    c = binding.Context(0)
    yield c
    c.close()


def _maxcut(n, seed):
    """min <-L/4, X> s.t. diag(X) = 1 for a seeded random graph with edge probability 0.3 (a stand-in for the
    public max-cut instances the paper's SDP runs use)."""
    u = inputs.rand((n, n), seed).numpy()
    A = np.triu((u < 0.3).astype(np.float64), 1)
    A = A + A.T
    return -0.25 * (np.diag(A.sum(1)) - A), np.ones(n)


def _rel(a, b):
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


@pytest.mark.parametrize("engine_name", ["fp32", "tf32", "half"])
def test_every_iteration_matches_the_oracle(ctx, engine_name):
    from paper_2609_21102_b200 import binding
    engine = binding.ENGINE_SIMT if engine_name == "fp32" else binding.ENGINE_AUTO
    n, K, k, sigma, warm = 256, 16, 6, 1.0, 2
    C, b = _maxcut(n, inputs.seed_for(5, 1, 7))
    V = np.linalg.qr(inputs.randn((n, K), inputs.seed_for(5, 1, inputs.PURPOSE_BASIS)).numpy())[0]
    v0 = inputs.gaussian_vector(n, 5, inputs.PURPOSE_LANCZOS).double().numpy()
    states = []
    st = {"V": V}

    def proj(Z, warmup):
        states.append({"V": st["V"].copy(), "Z": Z.copy(), "warm": warmup})
        P, Vn, _, _, _ = oracle.psd_project(Z, st["V"], k, SCHED, gamma=1.1, warmup=warmup, lanczos_v0=v0)
        st["V"] = Vn
        return P
    X, S = np.zeros((n, n)), np.zeros((n, n))
    Cd, bd = torch.tensor(C, dtype=torch.float32).cuda(), torch.tensor(b, dtype=torch.float32).cuda()
    v0d = torch.tensor(v0, dtype=torch.float32).cuda()
    for it in range(6):
        X1, S1, y1, res1 = oracle.admm_diag_sdp(C, b, sigma, 1, X, S, lambda Z, w: proj(Z, it < warm))
        Xd = torch.tensor(X, dtype=torch.float32).cuda()
        Sd = torch.tensor(S, dtype=torch.float32).cuda()
        Vd = torch.tensor(states[-1]["V"], dtype=torch.float32).cuda()
        yd, resd = ctx.defl_admm_diag_sdp(Cd, bd, sigma, 1, Xd, Sd, k, Vd, SCHED, warmup_iters=1 if it < warm else 0,
                                          gamma=1.1, lanczos_start=v0d, exploit_symmetry=True, engine=engine,
                                          half_filter=(engine_name == "half"))
        tol = TOL_ENGINE[engine_name]
        if engine_name in STORAGE:
            model, _ = storage_model.psd_storage_error(states[-1]["Z"], states[-1]["V"], k, SCHED, 1.1, states[-1]["warm"],
                                                       v0, STORAGE[engine_name])
            tol = min(tol, 2.0 * model + 1e-4)
            print("admm %s iteration %d: S error %.3e, storage model %.3e, tolerance %.3e" % (engine_name, it, _rel(Sd.cpu().double().numpy(), S1), model, tol))
        assert _rel(Sd.cpu().double().numpy(), S1) <= tol, (it, "S")
        # X_new = sigma (S - Z) is a difference of the projection and its argument: compared on the scale of S
        assert np.linalg.norm(Xd.cpu().double().numpy() - X1) <= tol * sigma * np.linalg.norm(S1), (it, "X")
        assert np.allclose(yd.cpu().double().numpy(), y1, atol=1e-5 * (1 + np.abs(y1).max()))      # no projection in y
        assert np.allclose(resd.double().numpy()[0], res1[0], atol=max(tol, 1e-3) * max(res1[0].max(), 1e-3) * 5), (it, resd, res1)
        assert _rel(Vd.cpu().double().numpy() @ Vd.cpu().double().numpy().T, st["V"] @ st["V"].T) <= 5e-2   # same subspace
        X, S = X1, S1


def test_residuals_are_what_the_iterates_say_and_fall(ctx):
    n, K, k, sigma = 384, 16, 6, 1.0
    C, b = _maxcut(n, inputs.seed_for(5, 2, 7))
    Cd, bd = torch.tensor(C, dtype=torch.float32).cuda(), torch.tensor(b, dtype=torch.float32).cuda()
    X, S = torch.zeros((n, n), device="cuda"), torch.zeros((n, n), device="cuda")
    V = inputs.randn((n, K), inputs.seed_for(5, 2, inputs.PURPOSE_BASIS)).float().cuda()
    y, res = ctx.defl_admm_diag_sdp(Cd, bd, sigma, 40, X, S, k, V, SCHED, warmup_iters=3, gamma=1.1, seed=5,
                                    exploit_symmetry=True)
    Xh, Sh, yh = X.cpu().double().numpy(), S.cpu().double().numpy(), y.cpu().double().numpy()
    want = [np.linalg.norm(np.diag(Xh) - b) / (1 + np.linalg.norm(b)),
            np.linalg.norm(np.diag(yh) + Sh - C) / (1 + np.linalg.norm(C)),
            abs(np.sum(C * Xh) - b @ yh) / (1 + abs(np.sum(C * Xh)) + abs(b @ yh))]
    assert np.allclose(res[-1].double().numpy(), want, rtol=1e-3, atol=1e-6)
    assert float(res[-1].max()) < 0.2 * float(res[0].max())
    assert torch.equal(S, S.T)


def test_kkt_point_stays_put(ctx):
    n, r, sigma = 128, 24, 1.0
    rng = np.random.default_rng(77)
    q, _ = np.linalg.qr(rng.standard_normal((n, n)))
    X = (q[:, :r] * rng.uniform(0.5, 2.0, r)) @ q[:, :r].T
    S = (q[:, r:] * rng.uniform(0.5, 2.0, n - r)) @ q[:, r:].T
    y = rng.standard_normal(n)
    C, b = S + np.diag(y), np.diag(X).copy()
    f = lambda a: torch.tensor(a, dtype=torch.float32).cuda()
    Xd, Sd = f(X), f(S)
    from paper_2609_21102_b200 import binding
    # exact fp32 products and 30 classical steps: the filter is the sign function on this spectrum (|x| >= 0.1)
    yd, res = ctx.defl_admm_diag_sdp(f(C), f(b), sigma, 2, Xd, Sd, 0, None, [list(oracle.CLASSICAL_QUINTIC)] * 30,
                                     exploit_symmetry=True, engine=binding.ENGINE_SIMT)
    assert _rel(Sd.cpu().double().numpy(), S) <= 1e-4
    assert np.linalg.norm(Xd.cpu().double().numpy() - X) <= 1e-4 * np.linalg.norm(S)
    assert np.allclose(yd.cpu().double().numpy(), y, atol=1e-4)
    assert float(res.max()) < 1e-4


def test_argument_errors(ctx):
    from paper_2609_21102_b200 import binding
    n = 30      # not a multiple of 4
    z = torch.zeros((n, n), device="cuda")
    with pytest.raises(binding.DeflError) as e:
        ctx.defl_admm_diag_sdp(z, torch.ones(n, device="cuda"), 1.0, 1, z.clone(), z.clone(), 0, None, SCHED)
    assert e.value.code == -1
