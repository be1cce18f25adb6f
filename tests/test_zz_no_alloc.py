"""isopo_layer_gram_static - the entry point for callers that cannot allocate device memory (a
hook running under a framework allocator that owns the device, or while that allocator is locked).
It keeps its scratch in a fixed array inside the library, so three things need checking through the
C ABI: that it returns what isopo_layer_gram returns on the Gram route (and what the fp64 oracle
defines K to be), that a second call, which finds the first call's leftovers in that shared array,
is still right, and that a call really allocates nothing on the device.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.  Passes alone in a fresh process and after the rest of the suite."""

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


def _problem(Ls, d_in, d_out, dtype, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    off = np.concatenate([[0], np.cumsum(Ls)]).astype(np.int64)
    T = int(off[-1])
    X = torch.randn(T, d_in, device="cuda", generator=g).to(dtype)
    dY = (0.1 * torch.randn(T, d_out, device="cuda", generator=g)).to(dtype)
    return X, dY, off


def _existing(b, X, dY, off):
    B = len(off) - 1
    code = b.BF16 if X.dtype == torch.bfloat16 else b.F32
    ws = b.alloc_workspace(code, X.shape[0], X.shape[1], dY.shape[1], B, b.PATH_GRAM)
    K = torch.empty(B, B, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.isopo_layer_gram(X, dY, off, K, ws, info, b.PATH_GRAM)
    torch.cuda.synchronize()
    assert int(info.item()) == 0
    return K


def _rel(a, ref):
    return float(torch.linalg.norm(a.double() - ref.double()) / torch.linalg.norm(ref.double()))


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 1e-5), (torch.bfloat16, 2e-2)])
def test_static_scratch_matches_workspace_entry_point_twice(b, dtype, tol):
    # first a larger problem, then a smaller one with other boundaries: stale offsets, map entries
    # or accumulators left in the shared array by call one would corrupt call two
    problems = [_problem([300, 17, 129, 64, 1, 250, 90], 72, 40, dtype, 1),
                _problem([40, 33, 200], 72, 40, dtype, 2)]
    for X, dY, off in problems:
        B = len(off) - 1
        want = _existing(b, X, dY, off)
        K = torch.full((B, B), float("nan"), device="cuda")
        info = torch.zeros(1, dtype=torch.int32, device="cuda")
        b.isopo_layer_gram_static(X, dY, off, K, info)
        torch.cuda.synchronize()
        assert int(info.item()) == 0
        assert torch.equal(K, K.T)
        assert _rel(K, want) <= tol
        # and against the definition itself: K_ij = <G_i, G_j> with every G_i materialised in float64
        K_o = orc.ntk(orc.sequence_gradients(to_f64(X), to_f64(dY), off))
        assert rel_fro(K.cpu().numpy(), K_o) <= tol


def test_static_scratch_call_allocates_nothing(b):
    """After one warm-up call (module load, symbol look-up), a further call must leave the device's free
    memory and torch's allocator exactly as they were - also with event timing switched on, which the
    call suspends for its duration because creating events allocates: its launches are counted, but no
    event is recorded for them."""
    X, dY, off = _problem([120, 40, 77], 64, 48, torch.bfloat16, 9)
    K = torch.empty(3, 3, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.isopo_layer_gram_static(X, dY, off, K, info)
    torch.cuda.synchronize()
    b.isopo_profile_enable(True)
    try:
        b.isopo_profile_collect()                      # forget whatever earlier tests left
        free0, _ = torch.cuda.mem_get_info()
        alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
        b.isopo_layer_gram_static(X, dY, off, K, info)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0
        assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
        prof = b.isopo_profile_collect()
        assert sum(n for _, n in prof.values()) >= 2   # prep + Gram kernel were launched and counted ...
        assert all(ms == 0.0 for ms, _ in prof.values())   # ... without an event pair around them
    finally:
        b.isopo_profile_enable(False)
    assert int(info.item()) == 0


def test_static_scratch_rejects_sizes_beyond_its_array(b):
    X = torch.zeros(8, 8, device="cuda")
    off_big_B = np.arange(b.STATIC_MAX_SEQS + 2, dtype=np.int64)
    Xb = torch.zeros(b.STATIC_MAX_SEQS + 1, 8, device="cuda")
    K = torch.empty((b.STATIC_MAX_SEQS + 1) ** 2, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(b.IsopoError) as e:
        b.isopo_layer_gram_static(Xb, Xb, off_big_B, K, info)
    assert e.value.status == b.ERR_UNSUPPORTED and "ISOPO_STATIC_MAX" in str(e.value)
    # too many tokens: rejected on the host before anything is read
    fake_T = b.STATIC_MAX_TOKENS + 1
    off = np.array([0, fake_T], dtype=np.int64)
    st = b.lib.isopo_layer_gram_static(X.data_ptr(), X.data_ptr(), b.F32, fake_T, 8, 8, off.ctypes.data, 1,
                                       K.data_ptr(), info.data_ptr(), None)
    assert st == b.ERR_UNSUPPORTED
