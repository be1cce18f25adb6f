"""Every mbarrier wait in the tensor-core kernels is bounded: after its clock limit the waiting role
raises the CTA's abort flag, records ISOPO_INFO_TIMEOUT | kernel id in *info, and all roles fall
through to the common teardown.  isopo_selftest_bounded_wait runs that very wait on a barrier that
nothing arrives on (no TMA, no tensor memory involved), so the path is exercised without hanging
or faulting anything; the context must be fully usable afterwards."""

import time

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


def test_wait_runs_out_and_the_library_still_works(b):
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    roles = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    b.isopo_selftest_bounded_wait(100_000, info, roles)
    torch.cuda.synchronize()
    elapsed = time.perf_counter() - t0
    probe_id = [k for k in range(b.NUM_KERNELS) if b.lib.isopo_kernel_name(k) == b"k_wait_probe"][0]
    assert int(info.item()) == (b.INFO_TIMEOUT | probe_id)
    assert int(roles.item()) == 3            # the role that gave up, the one released by the abort flag, the one without waits
    assert elapsed < 0.5                     # the second role did not sit out its own (one-second) limit

    # *info is only ever written over a zero: a second time-out leaves the first record in place
    info.fill_(5)
    b.isopo_selftest_bounded_wait(50_000, info, roles)
    torch.cuda.synchronize()
    assert int(info.item()) == 5 and int(roles.item()) == 3

    # the context is intact: a tensor-core call right after it matches the oracle
    g = torch.Generator(device="cuda")
    g.manual_seed(3)
    Ls = [70, 130, 64, 257]
    off = np.concatenate([[0], np.cumsum(Ls)]).astype(np.int64)
    X = torch.randn(int(off[-1]), 256, device="cuda", generator=g).to(torch.bfloat16)
    dY = (0.1 * torch.randn(int(off[-1]), 256, device="cuda", generator=g)).to(torch.bfloat16)
    A = torch.randn(4, device="cuda", generator=g)
    K_o, c_o, dW_o = orc.isopo_layer(to_f64(X), to_f64(dY), off, to_f64(A), orc.NORMALISED, 0.0)
    for path in (b.PATH_MATERIALISE, b.PATH_GRAM):
        res = b.isopo_layer(X, dY, off, A, b.VAR_NORMALISED, 0.0, path)
        assert res.info == 0
        assert rel_fro(res.K.cpu().numpy(), K_o) <= 2e-2
        assert rel_fro(res.dW.cpu().numpy(), dW_o) <= 2e-2


def test_limit_is_validated(b):
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    roles = torch.zeros(1, dtype=torch.int32, device="cuda")
    for bad in (0, -5, (1 << 28) + 1):
        with pytest.raises(b.IsopoError):
            b.isopo_selftest_bounded_wait(bad, info, roles)
