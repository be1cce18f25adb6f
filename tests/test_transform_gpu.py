"""GPU parity of isopo_transform_advantages alone: random Gram matrices of every block shape the
blocked Cholesky meets (B below, at and above multiples of 32, up to the 256 limit)."""

import numpy as np
import pytest
import torch

from oracle import isopo_oracle as orc
from tests._util import VARIANT_NAME, rel_fro

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2512_23353_b200 import binding
    return binding


def _gram(B, rank_extra, seed):
    """K = J J^T in float32 with strongly overlapping rows (a shared low-rank part)."""
    rng = np.random.default_rng(seed)
    J = rng.standard_normal((B, 4 * B + 8)) + 2.0 * rng.standard_normal((B, rank_extra)) @ rng.standard_normal((rank_extra, 4 * B + 8))
    K = (J @ J.T).astype(np.float32)
    return np.ascontiguousarray((K + K.T) / 2)


@pytest.mark.parametrize("B", [1, 2, 31, 32, 33, 64, 100, 200, 255, 256])
def test_interacting_solve(b, B):
    K = _gram(B, 3, B)
    A = np.random.default_rng(B + 1).standard_normal(B).astype(np.float32)
    for rel in (1e-3, 1.0):
        lam = np.float32(rel * np.mean(np.diag(K)))
        Kd, Ad = torch.from_numpy(K).cuda(), torch.from_numpy(A).cuda()
        c = torch.empty(B, device="cuda")
        info = torch.zeros(1, dtype=torch.int32, device="cuda")
        b.isopo_transform_advantages(Kd, Ad, b.VAR_INTERACTING, float(lam), c, info)
        torch.cuda.synchronize()
        assert int(info.item()) == 0
        want = orc.transform_advantages(K.astype(np.float64), A.astype(np.float64), orc.INTERACTING, float(lam))
        cond = np.linalg.cond(K.astype(np.float64) + float(lam) * np.eye(B))
        # float32 storage of c (6e-8) plus a refined float32 factorisation: far below 1e-5 for these conditions
        assert rel_fro(c.cpu().numpy(), want) <= max(1e-6, 1e-9 * cond), (B, rel, cond, rel_fro(c.cpu().numpy(), want))


@pytest.mark.parametrize("B", [5, 64, 256, 300, 1000])
def test_simple_variants_any_B(b, B):
    K = _gram(B, 2, 7 * B)
    A = np.random.default_rng(B).standard_normal(B).astype(np.float32)
    Kd, Ad = torch.from_numpy(K).cuda(), torch.from_numpy(A).cuda()
    lam = float(np.float32(0.01 * np.mean(np.diag(K))))
    for variant, g in ((b.VAR_NORMALISED, None), (b.VAR_NORMALISED_RAW, None), (b.VAR_DIRECTION, None),
                       (b.VAR_EUCLID, None), (b.VAR_REINFORCE, None), (b.VAR_GENERAL, [-1.0, 0.5, -2.0, lam, 0.0, 0.1])):
        c = torch.empty(B, device="cuda")
        info = torch.zeros(1, dtype=torch.int32, device="cuda")
        lam_v = 1e-3 if variant == b.VAR_DIRECTION else lam
        b.isopo_transform_advantages(Kd, Ad, variant, lam_v, c, info, g)
        torch.cuda.synchronize()
        pqr, regs = (tuple(g[:3]), tuple(np.float32(g[3:]).astype(np.float64))) if g else (None, None)
        want = orc.transform_advantages(K.astype(np.float64), A.astype(np.float64), VARIANT_NAME[variant],
                                        float(np.float32(lam_v)), pqr, regs)
        assert rel_fro(c.cpu().numpy(), want) <= 1e-6, (B, variant)


def test_not_pd_pivot_index_in_a_later_block(b):
    B = 70
    K = _gram(B, 2, 3).astype(np.float64)
    K[40, 40] = -1.0  # leading minor of order 41 is not positive definite
    Kd = torch.from_numpy(K.astype(np.float32)).cuda()
    c = torch.empty(B, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.isopo_transform_advantages(Kd, torch.ones(B, device="cuda"), b.VAR_INTERACTING, 0.0, c, info)
    torch.cuda.synchronize()
    assert int(info.item()) == 41


def test_relative_regulariser_runs_without_host_values(b):
    """gram -> isopo_reg_ema_update -> isopo_transform_advantages_rel over three microbatches: the
    running means and the coefficients must equal the oracle's, which is handed the same K matrices."""
    rng = np.random.default_rng(3)
    B = 48
    state = torch.zeros(4, device="cuda")
    o_state = (np.zeros(3), 0)
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    for step in range(3):
        M = rng.standard_normal((B, 300)) * (1.0 + step)
        K64 = M @ M.T
        K = torch.from_numpy(K64.astype(np.float32)).cuda()
        A = torch.from_numpy(rng.standard_normal(B).astype(np.float32)).cuda()
        K64 = K.double().cpu().numpy()
        b.isopo_reg_ema_update(K, 0.9, state)
        o_state = orc.ema_update(o_state, orc.regulariser_means(K64), 0.9)
        np.testing.assert_allclose(state[:3].cpu().numpy(), o_state[0], rtol=2e-6)
        assert int(state[3].item()) == step + 1
        for variant, name, idx in ((b.VAR_NORMALISED, orc.NORMALISED, 0), (b.VAR_DIRECTION, orc.DIRECTION, 2),
                                   (b.VAR_EUCLID, orc.EUCLID, 1), (b.VAR_INTERACTING, orc.INTERACTING, 1)):
            c = torch.empty(B, device="cuda")
            b.isopo_transform_advantages_rel(K, A, variant, 0.5, state, c, info)
            want = orc.transform_advantages(K64, A.double().cpu().numpy(), name, 0.5 * o_state[0][idx])
            assert rel_fro(c.cpu().numpy(), want) <= 1e-5, (step, name)
        g = [-1.0, -0.5, 0.25, 0.5, 2.0, 0.1]
        c = torch.empty(B, device="cuda")
        b.isopo_transform_advantages_rel(K, A, b.VAR_GENERAL, 0.0, state, c, info, g)
        want = orc.transform_advantages(K64, A.double().cpu().numpy(), orc.GENERAL, 0.0, tuple(g[:3]),
                                        (g[3] * o_state[0][0], g[4] * o_state[0][1], g[5] * o_state[0][2]))
        assert rel_fro(c.cpu().numpy(), want) <= 1e-5
    assert int(info.item()) == 0


@pytest.mark.parametrize("B,n", [(96, 7), (256, 7), (33, 32)])
def test_batched_layers_equal_single_calls_and_the_oracle(b, B, n):
    """One launch for n layers (different K and regulariser each, shared advantages) against the
    oracle per layer, and bit-for-bit against n single calls (the same kernel, one CTA per layer)."""
    A = np.random.default_rng(B).standard_normal(B).astype(np.float32)
    Ad = torch.from_numpy(A).cuda()
    Ks = [_gram(B, 1 + l % 4, 100 * B + l) * np.float32(1.0 + l) for l in range(n)]
    Kd = [torch.from_numpy(K).cuda() for K in Ks]
    lams = [float(np.float32((1e-3 if l % 2 else 0.3) * np.mean(np.diag(K)))) for l, K in enumerate(Ks)]
    for variant, name in ((b.VAR_INTERACTING, orc.INTERACTING), (b.VAR_NORMALISED, orc.NORMALISED)):
        info = torch.zeros(1, dtype=torch.int32, device="cuda")
        cs = [torch.full((B,), float("nan"), device="cuda") for _ in range(n)]
        b.isopo_transform_advantages_batched(Kd, Ad, variant, lams, cs, info)
        singles = [torch.empty(B, device="cuda") for _ in range(n)]
        for l in range(n):
            b.isopo_transform_advantages(Kd[l], Ad, variant, lams[l], singles[l], info)
        torch.cuda.synchronize()
        assert int(info.item()) == 0
        for l in range(n):
            assert torch.equal(cs[l], singles[l]), (name, l)
            want = orc.transform_advantages(Ks[l].astype(np.float64), A.astype(np.float64), name, lams[l])
            cond = np.linalg.cond(Ks[l].astype(np.float64) + lams[l] * np.eye(B)) if name == orc.INTERACTING else 1.0
            assert rel_fro(cs[l].cpu().numpy(), want) <= max(1e-6, 1e-9 * cond), (name, l, cond)


def test_batched_relative_regulariser_and_pivot_report(b):
    rng = np.random.default_rng(11)
    B, n = 40, 3
    Ks, states, o_lams = [], [], []
    for l in range(n):
        M = rng.standard_normal((B, 200)) * (1.0 + l)
        K = torch.from_numpy((M @ M.T).astype(np.float32)).cuda()
        st = torch.zeros(4, device="cuda")
        b.isopo_reg_ema_update(K, 0.9, st)
        Ks.append(K)
        states.append(st)
        o_lams.append(orc.regulariser_means(K.double().cpu().numpy())[1])  # E[K_ii]: the interacting variant's mean
    A = torch.from_numpy(rng.standard_normal(B).astype(np.float32)).cuda()
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    cs = [torch.empty(B, device="cuda") for _ in range(n)]
    factors = [0.5, 1.0, 0.25]
    b.isopo_transform_advantages_batched(Ks, A, b.VAR_INTERACTING, factors, cs, info, states=states)
    torch.cuda.synchronize()
    assert int(info.item()) == 0
    for l in range(n):
        want = orc.transform_advantages(Ks[l].double().cpu().numpy(), A.double().cpu().numpy(), orc.INTERACTING,
                                        factors[l] * o_lams[l])
        assert rel_fro(cs[l].cpu().numpy(), want) <= 1e-5, l
    # layer 1 is made indefinite at row 7: the report names the layer and the 1-based pivot
    bad = Ks[1].clone()
    bad[6, 6] = -1.0
    b.isopo_transform_advantages_batched([Ks[0], bad, Ks[2]], A, b.VAR_INTERACTING, [0.0, 0.0, 0.0], cs, info)
    torch.cuda.synchronize()
    assert int(info.item()) == 7 + (1 << 16)
    assert float(cs[1].abs().max().item()) == 0.0


def test_batched_argument_checks(b):
    B = 8
    K = torch.eye(B, device="cuda")
    A = torch.ones(B, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    c = torch.empty(B, device="cuda")
    with pytest.raises(b.IsopoError):
        b.isopo_transform_advantages_batched([K] * 33, A, b.VAR_NORMALISED, [0.1] * 33, [c] * 33, info)
    with pytest.raises(b.IsopoError):
        b.isopo_transform_advantages_batched([K], A, b.VAR_NORMALISED, [-1.0], [c], info)
    with pytest.raises(b.IsopoError):
        b.isopo_transform_advantages_batched([K], A, b.VAR_GENERAL, [0.0], [c], info)
