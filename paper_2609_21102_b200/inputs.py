"""Seeded synthetic inputs shared by the tests, the benchmark and the oracle checks.

This module only *makes matrices*: Haar-distributed orthogonal factors, prescribed spectra,
Gaussian bulks with planted spikes, a slowly drifting symmetric sequence and Gaussian sketches.
It contains none of the filter's arithmetic. Everything is generated in float64 from a
``torch.Generator`` seeded per (workload, shape, purpose, matrix index) and rounded once to the
storage type; the rounded values are what both the CUDA library and the CPU oracle read.

The five workloads mirror the shapes of GPT-2 small / medium / large / XL weight matrices and a
head-dominated symmetric matrix of SDP size. They stand in for recorded momentum matrices and for
public SDP instances, which are not available offline.
"""
import math

import torch

BASE_SEED = 260921102000
PURPOSE_MATRIX, PURPOSE_SKETCH, PURPOSE_LANCZOS, PURPOSE_BASIS = 0, 1, 2, 3


def seed_for(workload, shape_index=0, purpose=PURPOSE_MATRIX, index=0):
    return BASE_SEED + 100 * workload + 10 * shape_index + purpose + 1000003 * index


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def randn(shape, seed, device="cpu"):
    return torch.randn(shape, generator=_gen(seed, device), dtype=torch.float64, device=device)


def rand(shape, seed, device="cpu"):
    return torch.rand(shape, generator=_gen(seed, device), dtype=torch.float64, device=device)


def haar(rows, cols, seed, device="cpu"):
    """rows x cols matrix with orthonormal columns, Haar distributed (QR of a Gaussian, R's diagonal made positive)."""
    q, r = torch.linalg.qr(randn((rows, cols), seed, device))
    return q * torch.sign(torch.diagonal(r)).unsqueeze(0)


def from_spectrum(m, n, sigma, seed, device="cpu"):
    """U diag(sigma) V^T with Haar factors; len(sigma) = min(m, n)."""
    r = min(m, n)
    sigma = torch.as_tensor(sigma, dtype=torch.float64, device=device)
    u = haar(m, r, seed, device)
    v = haar(n, r, seed + 500009, device)
    return (u * sigma.unsqueeze(0)) @ v.T


def spectrum_tiny(seed, device="cpu"):
    """Workload 1: four dominant values and 124 values log-uniform in [1e-3, 1]."""
    tail = 10.0 ** (-3.0 * rand((124,), seed, device))
    head = torch.tensor([100.0, 50.0, 30.0, 20.0], dtype=torch.float64, device=device)
    return torch.cat([head, torch.sort(tail, descending=True).values])


def spectrum_power(r, exponent, top, floor=0.0, device="cpu"):
    i = torch.arange(1, r + 1, dtype=torch.float64, device=device)
    return torch.clamp(top * i ** (-exponent), min=floor)


def workload_tiny(b=4, m=128, n=256, device="cpu"):
    """Workload 1 (fp32): b matrices m x n = U diag(s) V^T."""
    mats = [from_spectrum(m, n, spectrum_tiny(seed_for(1, 0, 0, i) + 7, device), seed_for(1, 0, 0, i), device)
            for i in range(b)]
    return torch.stack(mats)


def workload_spiked(b, m, n, shape_index, spikes=8, factor=30.0, device="cpu"):
    """Workload 2: N(0,1) bulk plus `spikes` rank-one terms u_i v_i^T of size factor * ||N||_F / sqrt(n)."""
    out = []
    for i in range(b):
        sd = seed_for(2, shape_index, 0, i)
        bulk = randn((m, n), sd, device)
        u = haar(m, spikes, sd + 11, device)
        v = haar(n, spikes, sd + 13, device)
        s = factor * torch.linalg.norm(bulk) / math.sqrt(n)
        out.append(bulk + s * (u @ v.T))
    return torch.stack(out)


def workload_power_law(b, m, n, workload, shape_index, exponent, top, floor=0.0, device="cpu"):
    """Workloads 3 and 4: sigma_i = max(top * i^-exponent, floor) with Haar factors."""
    sig = spectrum_power(min(m, n), exponent, top, floor, device)
    return torch.stack([from_spectrum(m, n, sig, seed_for(workload, shape_index, 0, i), device) for i in range(b)])


def sdp_spectrum(n, heads=8, head_mag=1.0e3, seed=None, device="cpu"):
    seed = seed_for(5, 0, 0, 0) if seed is None else seed
    signs = torch.where(rand((heads,), seed + 3, device) < 0.5, -1.0, 1.0).to(torch.float64)
    bulk = 2.0 * rand((n - heads,), seed + 5, device) - 1.0
    return torch.cat([head_mag * signs, bulk])


def sdp_first(n, heads=8, head_mag=1.0e3, device="cpu"):
    """Workload 5, first iterate: Q diag(lambda) Q^T with `heads` eigenvalues +-head_mag and the rest uniform in [-1, 1]."""
    lam = sdp_spectrum(n, heads, head_mag, device=device)
    q = haar(n, n, seed_for(5, 0, 0, 0), device)
    x = (q * lam.unsqueeze(0)) @ q.T
    return 0.5 * (x + x.T), lam


def sdp_next(x, t, step=1.0e-3):
    """Workload 5, drift: X_{t+1} = X_t + step * sym(N(0,1))."""
    nse = randn(tuple(x.shape), seed_for(5, 0, 0, t), x.device)
    return x + step * 0.5 * (nse + nse.T)


def sketch(b, ms, l, workload, shape_index=0, device="cpu"):
    """Gaussian sketch Omega[b, ms, l], float32 (Algorithm 3 draws it; here it is an explicit input)."""
    return randn((b, ms, l), seed_for(workload, shape_index, PURPOSE_SKETCH), device).to(torch.float32)


def gaussian_vector(n, workload, purpose, index=0, device="cpu"):
    return randn((n,), seed_for(workload, 0, purpose, index), device).to(torch.float32)


def round_to(x, dtype):
    """Round a float64 tensor once to the storage type."""
    return x.to(dtype)
