"""GPU parity at the ends of the size ranges: millions of tokens, a single token, 2048 single-token sequences, sequence
counts on both sides of the weight-gradient kernels' on-chip limit (2048), one sequence of half a million tokens, the
widest and the narrowest layers of the 7B-class block.  K (Algorithm 2, "make neural tangent kernel") and dW = sum_i
c_i G_i against the oracle; tolerances 2e-2 (bfloat16) and 1e-5 (float32) in relative Frobenius norm."""

import numpy as np
import pytest
import torch

from oracle import isopo_oracle as orc
from tests._util import rel_fro, report, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2512_23353_b200 import binding
    return binding


def _lengths(kind):
    rng = np.random.default_rng(5150)
    return {
        "3M tokens": rng.integers(30000, 60000, size=64).tolist(),
        "one token": [1],
        "2048 single tokens": [1] * 2048,
        "2048 sequences": rng.integers(96, 200, size=2048).tolist(),
        "2049 sequences": [100] * 2049,
        "one long sequence": [500000],
        "three": [300, 200, 100],
    }[kind]


CASES = [
    # (name, lengths, d_in, d_out, dtype, paths for K ("stored" / "gram"))
    ("3M tokens, narrow bf16 layer", "3M tokens", 8, 8, torch.bfloat16, ("stored",)),
    ("3M tokens, narrow f32 layer", "3M tokens", 16, 8, torch.float32, ("stored",)),
    ("one token", "one token", 8, 8, torch.bfloat16, ("stored", "gram")),
    ("2048 single-token sequences", "2048 single tokens", 64, 64, torch.bfloat16, ("gram",)),
    ("2048 sequences: the most the fold kernel stages", "2048 sequences", 256, 256, torch.bfloat16, ()),
    ("2049 sequences: one more", "2049 sequences", 256, 256, torch.bfloat16, ()),
    ("one sequence of 500k tokens", "one long sequence", 264, 520, torch.bfloat16, ("stored",)),
    ("8 -> 18944", "three", 8, 18944, torch.bfloat16, ("stored", "gram")),
    ("18944 -> 8", "three", 18944, 8, torch.bfloat16, ("stored", "gram")),
]


@pytest.mark.parametrize("case", range(len(CASES)))
def test_extreme_size_matches_oracle(b, case):
    name, kind, d_in, d_out, dtype, paths = CASES[case]
    Ls = _lengths(kind)
    off = np.concatenate([[0], np.cumsum(Ls)]).astype(np.int64)
    T, B = int(off[-1]), len(Ls)
    tol = 2e-2 if dtype == torch.bfloat16 else 1e-5
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5200 + case)
    X = torch.randn(T, d_in, device="cuda", generator=gen).to(dtype)
    dY = (0.1 * torch.randn(T, d_out, device="cuda", generator=gen)).to(dtype)
    A = torch.from_numpy(np.random.default_rng(5300 + case).standard_normal(B).astype(np.float32)).cuda()
    G = orc.sequence_gradients(to_f64(X), to_f64(dY), off)
    errs = {}
    if paths:
        K_o = orc.ntk(G)
        lam = 1e-3 * float(np.mean(np.diag(K_o)))
        for pname in paths:
            res = b.isopo_layer(X, dY, off, A, b.VAR_NORMALISED, lam, b.PATH_MATERIALISE if pname == "stored" else b.PATH_GRAM)
            torch.cuda.synchronize()
            assert res.info == 0, (name, pname, hex(res.info))
            errs[f"K_{pname}"] = rel_fro(res.K.cpu().numpy(), K_o)
            errs[f"dW_{pname}"] = rel_fro(res.dW.cpu().numpy(), orc.weight_gradient(G, to_f64(res.coeffs)))
    # the weight gradient alone on the GEMM route (dispatch between its three kernels)
    ws = b.alloc_workspace(b.BF16 if dtype == torch.bfloat16 else b.F32, T, d_in, d_out, B, b.PATH_GRAM)
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    dW = torch.empty(d_out, d_in, device="cuda")
    b.isopo_weight_grad(X, dY, A, off, dW, ws, info, b.PATH_GRAM, 0.0)
    torch.cuda.synchronize()
    assert int(info.item()) == 0, name
    errs["dW_gemm_route"] = rel_fro(dW.cpu().numpy(), orc.weight_gradient(G, to_f64(A)))
    report(f"{name}: T={T} B={B} {d_in}->{d_out}", **errs)
    assert all(e <= tol for e in errs.values()), (name, errs)
