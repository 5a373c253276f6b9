"""Seeded random shapes and options through defl_polar_batched against the oracle: ragged and aligned sizes, tall and
wide, k = 0 and k > 0, J = 0..2, L = 1..6, both storage types, symmetric tiles on and off. PADDED restore only:
Eq. 3's post-add (ADD mode) amplifies the difference between two inexact sets of triplets by a^L, which is a
property of that mode (the paper pads for this reason), not of an implementation."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_21102_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2609_21102_b200 import binding
    c = binding.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_configurations(ctx, seed):
    from paper_2609_21102_b200 import binding
    rng = np.random.default_rng(seed)
    mu = list(binding.MUON_QUINTIC)
    for trial in range(12):
        b = int(rng.integers(1, 5))
        m, n = int(rng.integers(24, 720)), int(rng.integers(24, 720))
        if rng.random() < 0.5:                      # half of the cases on sizes the tensor engine takes
            m, n = (m // 8) * 8 + 8, (n // 8) * 8 + 8
        ms = min(m, n)
        k = int(rng.integers(0, min(12, ms // 3)))
        p = int(rng.integers(2, 9)) if k else 0
        J, L, sym = int(rng.integers(0, 3)), int(rng.integers(1, 7)), bool(rng.integers(0, 2))
        dt = torch.bfloat16 if rng.random() < 0.75 else torch.float32
        l = min(ms, k + p)
        # a head of k values in [5, 60] over a bulk in [0.05, 1]: the gap makes the window well defined
        sigma = np.concatenate([np.sort(rng.uniform(5, 60, max(k, 1)))[::-1], rng.uniform(0.05, 1.0, ms - max(k, 1))])
        G = torch.stack([inputs.from_spectrum(m, n, sigma, 7000 * seed + 10 * trial + i) for i in range(b)]).to(dt)
        Om = torch.tensor(rng.standard_normal((b, ms, max(l, 1))), dtype=torch.float32)
        out, info = ctx.defl_polar_batched(G.cuda(), k, p, J, [mu] * L, sketch=Om.cuda() if k else None, gamma=1.05,
                                           exploit_symmetry=sym, want_info=True)
        torch.cuda.synchronize()
        case = (seed, trial, b, m, n, k, p, J, L, sym, str(dt))
        assert int(info["status"].max()) == 0, case
        tol = 3e-2 if dt == torch.bfloat16 else 2e-3
        for i in range(b):
            ref, *_ = oracle.deflated_polar(G[i].double().numpy(), k, l, Om[i].double().numpy(), J,
                                            oracle.schedule([mu] * L), gamma=1.05)
            err = float(np.linalg.norm(out[i].double().cpu().numpy() - ref) / np.linalg.norm(ref))
            assert err <= tol, (case, i, err)
