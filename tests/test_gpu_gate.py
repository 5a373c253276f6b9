"""The deflation gate of Algorithms 1 and 2 (threshold tau), decided per matrix on the device, against the oracle."""
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


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 2e-3), (torch.bfloat16, 3e-2)])
@pytest.mark.parametrize("mode", [0, 1])
def test_polar_gate_per_matrix(ctx, dtype, tol, mode):
    m, n, k, p, J, tau = 160, 288, 6, 6, 2, 0.1
    tail = torch.linspace(1.0, 0.05, 160 - 3, dtype=torch.float64)
    spectra = [torch.cat([torch.tensor([60.0, 40.0, 25.0], dtype=torch.float64), tail]),     # gate fires, 3 of 6 deflated
               torch.linspace(2.0, 0.5, 160, dtype=torch.float64),                             # flat: gate stays off
               torch.cat([torch.tensor([90.0, 70.0, 50.0, 30.0, 20.0], dtype=torch.float64), tail[:-2]])]   # 5 of 6
    G = torch.stack([inputs.from_spectrum(m, n, s, 7000 + i) for i, s in enumerate(spectra)]).to(dtype).cuda()
    Om = inputs.sketch(3, m, k + p, 1).cuda()
    out, info = ctx.defl_polar_batched(G, k, p, J, [MUON] * 5, sketch=Om, gamma=1.01, restore_mode=mode, tau=tau,
                                       exploit_symmetry=True, want_info=True)
    torch.cuda.synchronize()
    assert info["k_used"].cpu().tolist() == [3, 0, 5]
    for i in range(3):
        ref, s, kk, rho = oracle.deflated_polar(G[i].double().cpu().numpy(), k, k + p, Om[i].double().cpu().numpy(), J,
                                                oracle.schedule([MUON] * 5), tau=tau, gamma=1.01, mode=mode)
        assert kk == int(info["k_used"][i])
        assert _rel(out[i].double().cpu().numpy(), ref) <= tol
        assert abs(float(info["rho"][i]) - rho) <= 2e-3 * rho
    # the matrix whose gate stayed off equals the plain filter of that matrix
    plain = ctx.defl_polar_batched(G[1:2].contiguous(), 0, 0, 0, [MUON] * 5, exploit_symmetry=True)
    assert _rel(out[1].double().cpu().numpy(), plain[0].double().cpu().numpy()) <= (1e-5 if dtype == torch.float32 else 2e-2)


def test_psd_gate(ctx):
    n, K, window, tau = 256, 8, 6, 0.1
    lam = torch.cat([torch.tensor([40.0, -35.0, 30.0], dtype=torch.float64), 2.0 * inputs.rand((n - 3,), 99) - 1.0])
    q = inputs.haar(n, n, 98)
    X64 = (q * lam.unsqueeze(0)) @ q.T
    X = (0.5 * (X64 + X64.T)).float().cuda()
    sched = [[1.875, -1.25, 0.375]] * 7
    v0 = inputs.gaussian_vector(n, 5, inputs.PURPOSE_LANCZOS, 3).cuda()
    # basis: the three dominant eigenvectors plus five bulk directions, so the Ritz pairs are sharp
    idx = [0, 1, 2, 10, 20, 30, 40, 50]
    V = q[:, idx].float().contiguous().cuda()
    Vo = V.double().cpu().numpy()
    qo, ro = np.linalg.qr(Vo)
    Vo = qo * np.sign(np.diag(ro))[None, :]
    P, info = ctx.defl_psd_project(X, window, V, sched, gamma=1.1, lanczos_start=v0, tau=tau, want_info=True)
    torch.cuda.synchronize()
    Po, _, lam_o, ndef, th = oracle.psd_project(X.double().cpu().numpy(), Vo, window, oracle.schedule(sched), tau=tau,
                                                gamma=1.1, lanczos_v0=v0.double().cpu().numpy())
    assert ndef == 3 and int(info["k_used"][0]) == 3
    assert _rel(P.double().cpu().numpy(), Po) <= 2e-3
    assert abs(float(info["theta"][0]) - th) <= 2e-3 * th
    # window of 2: |lambda_2| = 35 is not below tau * 40, the gate stays off and the call is the undeflated baseline
    V2 = q[:, idx].float().contiguous().cuda()
    P2, info2 = ctx.defl_psd_project(X, 2, V2, sched, gamma=1.1, lanczos_start=v0, tau=tau, want_info=True)
    Po2, _, _, ndef2, _ = oracle.psd_project(X.double().cpu().numpy(), Vo, 2, oracle.schedule(sched), tau=tau, gamma=1.1,
                                             lanczos_v0=v0.double().cpu().numpy())
    assert ndef2 == 0 and int(info2["k_used"][0]) == 0
    assert _rel(P2.double().cpu().numpy(), Po2) <= 2e-3
