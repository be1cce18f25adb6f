"""GPU parity of isopo_transform_spectral (Alg. 2's eigendecomposition route) against the oracle's
spectral form: coefficients, spectrum, the cut-off on a rank-deficient kernel, and agreement with the
Cholesky route of isopo_transform_advantages on the same K."""

import time

import numpy as np
import pytest
import torch

from oracle import isopo_oracle as orc
from tests._util import rel_fro

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2512_23353_b200 import binding
    return binding


def _gram(B, rank_extra, seed):
    rng = np.random.default_rng(seed)
    J = rng.standard_normal((B, 4 * B + 8)) + 2.0 * rng.standard_normal((B, rank_extra)) @ rng.standard_normal((rank_extra, 4 * B + 8))
    K = (J @ J.T).astype(np.float32)
    return np.ascontiguousarray((K + K.T) / 2)


@pytest.mark.parametrize("B", [1, 2, 5, 33, 64, 127, 200, 256])
def test_coefficients_and_spectrum(b, B):
    K = _gram(B, 3, 50 + B)
    A = np.random.default_rng(B).standard_normal(B).astype(np.float32)
    lam = float(np.float32(1e-3 * np.mean(np.diag(K))))
    Kd, Ad = torch.from_numpy(K).cuda(), torch.from_numpy(A).cuda()
    c, eig = torch.empty(B, device="cuda"), torch.empty(B, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.isopo_transform_spectral(Kd, Ad, lam, c, info, eigenvalues=eig)
    torch.cuda.synchronize()
    assert int(info.item()) == 0
    c_o, D_o = orc.spectral_coefficients(K.astype(np.float64), A.astype(np.float64), lam)
    cond = (D_o[0] + lam) / (max(D_o[-1], 0.0) + lam)
    # float32 columns, float64 inner products: eigenvalues to a few ulp of the largest one
    assert np.max(np.abs(eig.cpu().numpy() - D_o)) <= 2e-6 * D_o[0]
    assert np.all(np.diff(eig.cpu().numpy()) <= 0)
    # a float32 eigenbasis: error of the solve about eps_f32 * cond
    tol = 1e-5 + 1e-7 * cond
    assert rel_fro(c.cpu().numpy(), c_o) <= tol, (B, cond, rel_fro(c.cpu().numpy(), c_o))
    # the Cholesky route on the same K
    c2 = torch.empty(B, device="cuda")
    b.isopo_transform_advantages(Kd, Ad, b.VAR_INTERACTING, lam, c2, info)
    torch.cuda.synchronize()
    assert int(info.item()) == 0
    assert rel_fro(c.cpu().numpy(), c2.cpu().numpy()) <= tol


def test_cutoff_on_a_rank_deficient_kernel(b):
    """Every sequence twice: K has rank B / 2, the Cholesky route stops at a zero pivot with lambda = 0,
    the spectral route with the null directions cut off returns the minimum-norm solution."""
    half = _gram(20, 2, 7).astype(np.float64)
    K = np.block([[half, half], [half, half]]).astype(np.float32)
    A = np.random.default_rng(8).standard_normal(40).astype(np.float32)
    Kd, Ad = torch.from_numpy(K).cuda(), torch.from_numpy(A).cuda()
    c, eig = torch.empty(40, device="cuda"), torch.empty(40, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.isopo_transform_spectral(Kd, Ad, 0.0, c, info, rel_cutoff=1e-4, eigenvalues=eig)
    torch.cuda.synchronize()
    assert int(info.item()) == 0
    c_o, D_o = orc.spectral_coefficients(K.astype(np.float64), A.astype(np.float64), 0.0, 1e-4)
    e = eig.cpu().numpy()
    assert np.sum(e > 1e-4 * e[0]) == 20 and np.max(np.abs(e - D_o)) <= 2e-6 * D_o[0]
    cond = D_o[0] / D_o[19]
    # columns of K V shorter than 3e-7 ||K||_F are not rotated any further, so a kept direction can carry
    # that much of the null space relative to its own eigenvalue: 3e-7 sqrt(rank) d_max / d_min
    tol = 1e-5 + 3e-7 * np.sqrt(20.0) * cond
    assert rel_fro(c.cpu().numpy(), c_o) <= tol, (cond, rel_fro(c.cpu().numpy(), c_o))
    np.testing.assert_allclose(c.cpu().numpy()[:20], c.cpu().numpy()[20:], rtol=1e-3, atol=1e-6 * np.abs(c_o).max())


def test_time_at_full_size_and_argument_checks(b, capsys):
    K = _gram(256, 3, 1)
    Kd = torch.from_numpy(K).cuda()
    A = torch.ones(256, device="cuda")
    c = torch.empty(256, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    lam = float(1e-3 * np.mean(np.diag(K)))
    ws = torch.empty(b.lib.isopo_spectral_workspace_bytes(), dtype=torch.uint8, device="cuda")
    b.isopo_transform_spectral(Kd, A, lam, c, info, ws=ws)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    b.isopo_transform_spectral(Kd, A, lam, c, info, ws=ws)
    torch.cuda.synchronize()
    ms = (time.perf_counter() - t0) * 1e3
    with capsys.disabled():
        print(f"\n[isopo_transform_spectral, B = 256: {ms:.2f} ms]")
    assert int(info.item()) == 0 and ms < 100.0
    with pytest.raises(b.IsopoError):
        b.isopo_transform_spectral(Kd, A, -1.0, c, info, ws=ws)
    with pytest.raises(b.IsopoError):
        b.isopo_transform_spectral(Kd, A, lam, c, info, rel_cutoff=1.0, ws=ws)
    with pytest.raises(b.IsopoError):
        b.isopo_transform_spectral(Kd, A, lam, c, info, ws=ws[:1024])
    big = torch.eye(300, device="cuda")
    with pytest.raises(b.IsopoError):
        b.isopo_transform_spectral(big, torch.ones(300, device="cuda"), lam, torch.empty(300, device="cuda"), info)


def test_seven_layers_in_one_launch(b, capsys):
    """The block's seven K in one launch, one cluster per layer: the same results as seven calls, in
    about the time of one."""
    B, n = 256, 7
    Ks = [torch.from_numpy(_gram(B, 1 + l % 3, 900 + l) * np.float32(1 + l)).cuda() for l in range(n)]
    A = torch.from_numpy(np.random.default_rng(5).standard_normal(B).astype(np.float32)).cuda()
    lams = [float(1e-3 * torch.diagonal(K).mean().item()) for K in Ks]
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    cs = [torch.empty(B, device="cuda") for _ in range(n)]
    es = [torch.empty(B, device="cuda") if l % 2 == 0 else None for l in range(n)]
    b.isopo_transform_spectral_batched(Ks, A, lams, cs, info, eigenvalues=es)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    b.isopo_transform_spectral_batched(Ks, A, lams, cs, info, eigenvalues=es)
    torch.cuda.synchronize()
    ms = (time.perf_counter() - t0) * 1e3
    with capsys.disabled():
        print(f"\n[isopo_transform_spectral_batched, 7 x B = 256: {ms:.2f} ms]")
    assert int(info.item()) == 0
    for l in range(n):
        c1, e1 = torch.empty(B, device="cuda"), torch.empty(B, device="cuda")
        b.isopo_transform_spectral(Ks[l], A, lams[l], c1, info, eigenvalues=e1)
        torch.cuda.synchronize()
        assert torch.equal(c1, cs[l])
        if es[l] is not None:
            assert torch.equal(e1, es[l])
    assert int(info.item()) == 0
    with pytest.raises(b.IsopoError):
        b.isopo_transform_spectral_batched(Ks, A, lams, cs, info, ws=torch.empty(1024, dtype=torch.uint8, device="cuda"))
