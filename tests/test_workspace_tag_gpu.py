"""isopo_weight_grad on the materialised route sums whatever isopo_layer_gram left in the workspace.
The workspace carries a tag (dtype, T, d_in, d_out, B, a hash of the offsets); a call whose arguments
do not match it must leave dW alone and report ISOPO_INFO_STALE_WORKSPACE in *info, and the matching
call must still give Alg. 2's dW = sum_i c_i G_i."""

import numpy as np
import pytest
import torch

from oracle import isopo_oracle as orc
from tests._util import rel_fro, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2512_23353_b200 import binding
    return binding


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 1e-5), (torch.bfloat16, 2e-2)])
def test_stale_workspace_is_reported_and_dw_left_alone(b, dtype, tol):
    g = torch.Generator(device="cuda")
    g.manual_seed(5)
    Ls = [30, 50, 20, 28]
    off = np.concatenate([[0], np.cumsum(Ls)]).astype(np.int64)
    other = np.concatenate([[0], np.cumsum([31, 49, 20, 28])]).astype(np.int64)   # same T and B, other boundaries
    T, B, d_in, d_out = int(off[-1]), 4, 80, 40
    X = torch.randn(T, d_in, device="cuda", generator=g).to(dtype)
    dY = (0.1 * torch.randn(T, d_out, device="cuda", generator=g)).to(dtype)
    c = torch.tensor([0.5, -1.0, 2.0, 0.25], device="cuda")
    code = b.BF16 if dtype == torch.bfloat16 else b.F32
    ws = b.alloc_workspace(code, T, d_in, d_out, B, b.PATH_MATERIALISE)
    K = torch.empty(B, B, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.isopo_layer_gram(X, dY, off, K, ws, info, b.PATH_MATERIALISE)

    dW = torch.full((d_out, d_in), 7.0, device="cuda")
    b.isopo_weight_grad(X, dY, c, other, dW, ws, info, b.PATH_MATERIALISE, 0.0)
    torch.cuda.synchronize()
    assert int(info.item()) == b.INFO_STALE_WORKSPACE
    assert bool((dW == 7.0).all())

    # a layer of another shape whose workspace is no larger: rejected the same way
    info.zero_()
    dW2 = torch.full((d_out, d_in // 2), 7.0, device="cuda")
    X2 = X[:, : d_in // 2].contiguous()
    b.isopo_weight_grad(X2, dY, c, off, dW2, ws, info, b.PATH_MATERIALISE, 0.0)
    torch.cuda.synchronize()
    assert int(info.item()) == b.INFO_STALE_WORKSPACE
    assert bool((dW2 == 7.0).all())

    info.zero_()
    b.isopo_weight_grad(X, dY, c, off, dW, ws, info, b.PATH_MATERIALISE, 0.0)
    torch.cuda.synchronize()
    assert int(info.item()) == 0
    G = orc.sequence_gradients(to_f64(X), to_f64(dY), off)
    assert rel_fro(dW.cpu().numpy(), orc.weight_gradient(G, to_f64(c))) <= tol
