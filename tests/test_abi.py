"""Host-side checks of the C ABI: the library loads, exports every declared symbol, validates its
arguments before touching the GPU, and the path cost model behaves."""

import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2512_23353_b200 import build
    build.build()
    from paper_2512_23353_b200 import binding as b
    return b


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "isopo.h")).read()
    return sorted(set(re.findall(r"ISOPO_API[^;(]*?\b(isopo_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol(binding):
    declared = _declared_symbols()
    assert len(declared) >= 7
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in isopo.h but not exported"
    assert set(declared) == set(binding.EXPORTS)


def test_status_strings(binding):
    names = [binding.lib.isopo_status_string(i).decode() for i in range(5)]
    assert names == ["ISOPO_OK", "ISOPO_ERR_INVALID_ARG", "ISOPO_ERR_UNSUPPORTED", "ISOPO_ERR_WORKSPACE",
                     "ISOPO_ERR_CUDA"]
    assert binding.lib.isopo_status_string(99).decode() == "ISOPO_ERR_UNKNOWN"


def test_path_choice_follows_cost_model(binding):
    b = binding
    # LLM-length sequences: the token Gram costs (d_in+d_out) T^2, far above the stored-gradient route
    assert b.isopo_choose_path(b.BF16, 354_600, 1536, 8960, 256) == b.PATH_MATERIALISE
    assert b.isopo_choose_path(b.BF16, 294_900, 3584, 18944, 64) == b.PATH_MATERIALISE
    assert b.isopo_choose_path(b.BF16, 36_900, 896, 4864, 64) == b.PATH_MATERIALISE
    # short sequences on a wide layer: Gram wins
    assert b.isopo_choose_path(b.BF16, 2_000, 896, 4864, 32) == b.PATH_GRAM
    # more sequences than the stored-gradient kernels hold on chip
    assert b.isopo_choose_path(b.BF16, 100_000, 1024, 1024, 512) == b.PATH_GRAM
    # monotone in T
    prev = b.PATH_GRAM
    for T in (256, 1024, 4096, 16384, 65536, 262144):
        p = b.isopo_choose_path(b.BF16, T, 1024, 1024, 64)
        assert not (prev == b.PATH_MATERIALISE and p == b.PATH_GRAM)
        prev = p
    assert prev == b.PATH_MATERIALISE


def test_workspace_bytes(binding):
    b = binding
    assert b.isopo_workspace_bytes(b.BF16, 0, 64, 64, 1) == 0
    assert b.isopo_workspace_bytes(b.BF16, 10, 64, 64, 11) == 0
    gram = b.isopo_workspace_bytes(b.BF16, 4096, 1536, 8960, 16, b.PATH_GRAM)
    mat = b.isopo_workspace_bytes(b.BF16, 4096, 1536, 8960, 16, b.PATH_MATERIALISE)
    assert mat >= 2 * 16 * 1536 * 8960
    # Gram route: offsets, order, token map and the pre-scaled narrower operand of the weight-gradient GEMM
    assert 2 * 4096 * 1536 <= gram < 2 * 4096 * 1536 + (1 << 20)
    f32 = b.isopo_workspace_bytes(b.F32, 320, 64, 64, 8, b.PATH_MATERIALISE)
    assert f32 >= 4 * 8 * 64 * 64


def test_argument_validation_happens_on_the_host(binding):
    """Bad arguments are rejected before any CUDA call, so this runs without a GPU."""
    b = binding
    off = np.array([0, 3, 5], dtype=np.int64)
    fake = 1 << 20  # never dereferenced
    call = lambda **kw: b.lib.isopo_layer_gram(  # noqa: E731
        kw.get("X", fake), fake, kw.get("dtype", b.F32), kw.get("T", 5), kw.get("d_in", 8), 8,
        kw.get("off", off).ctypes.data, 2, kw.get("path", b.PATH_GRAM), fake, kw.get("ws", fake),
        kw.get("ws_bytes", 1 << 30), fake, None)
    assert call(X=None) == b.ERR_INVALID_ARG
    assert call(X=fake + 4) == b.ERR_INVALID_ARG                       # misaligned
    assert call(ws=fake + 512) == b.ERR_INVALID_ARG                    # workspace not 1024-aligned
    assert call(T=6) == b.ERR_INVALID_ARG                              # offsets do not end at T
    assert call(off=np.array([0, 5, 5], dtype=np.int64)) == b.ERR_INVALID_ARG   # empty sequence
    assert call(off=np.array([1, 3, 5], dtype=np.int64)) == b.ERR_INVALID_ARG
    assert call(path=7) == b.ERR_INVALID_ARG
    assert call(dtype=b.BF16, d_in=12) == b.ERR_UNSUPPORTED            # bf16 rows must be 16-byte multiples
    assert call(ws_bytes=16) == b.ERR_WORKSPACE
    tr = lambda B=4, variant=b.VAR_NORMALISED, lam=0.0, g=None: b.lib.isopo_transform_advantages(  # noqa: E731
        fake, fake, B, variant, lam, g, fake, fake, None)
    assert tr(B=0) == b.ERR_INVALID_ARG
    assert tr(variant=11) == b.ERR_INVALID_ARG
    assert tr(lam=-1.0) == b.ERR_INVALID_ARG
    assert tr(variant=b.VAR_GENERAL) == b.ERR_INVALID_ARG              # needs p, q, r and the regularisers
    assert tr(B=300, variant=b.VAR_INTERACTING) == b.ERR_UNSUPPORTED
    wg = b.lib.isopo_weight_grad(fake, fake, b.F32, 5, 8, 8, fake, off.ctypes.data, 2, b.PATH_GRAM, fake, 0.5,
                                 fake, 1 << 30, fake, None)
    assert wg == b.ERR_INVALID_ARG                                     # beta must be 0 or 1


def test_new_entry_points_validate_on_the_host(binding):
    """The entry points added around the three calls reject bad arguments before any CUDA call, and the
    process-wide switches change what they say they change (workspace size, nothing else)."""
    b = binding
    off = np.array([0, 3, 5], dtype=np.int64)
    fake = 1 << 20
    ptrs = np.array([fake, fake + (1 << 16), fake + (1 << 17)], dtype=np.uint64)
    widths = np.array([8, 8, 8], dtype=np.int32)
    sizes = np.array([1 << 30] * 3, dtype=np.uint64)
    stored = lambda **kw: b.lib.isopo_layer_gram_shared_x_stored(  # noqa: E731
        fake, kw.get("n", 2), ptrs.ctypes.data, widths.ctypes.data, kw.get("dtype", b.BF16), 5, 8, off.ctypes.data,
        kw.get("B", 2), ptrs.ctypes.data, kw.get("ws", ptrs).ctypes.data, kw.get("sizes", sizes).ctypes.data, fake, None)
    assert stored(n=0) == b.ERR_INVALID_ARG and stored(n=4) == b.ERR_INVALID_ARG
    assert stored(dtype=b.F32) == b.ERR_UNSUPPORTED
    assert stored(ws=np.array([fake, fake, fake], dtype=np.uint64)) == b.ERR_INVALID_ARG      # one workspace twice
    assert stored(sizes=np.array([16, 16, 16], dtype=np.uint64)) == b.ERR_WORKSPACE
    assert b.lib.isopo_selftest_bounded_wait(0, fake, fake, None) == b.ERR_INVALID_ARG
    assert b.lib.isopo_selftest_bounded_wait(1000, None, fake, None) == b.ERR_INVALID_ARG
    assert b.lib.isopo_set_store_format(5) == b.ERR_INVALID_ARG
    assert b.lib.isopo_get_store_format() == b.STORE_BF16
    base = b.isopo_workspace_bytes(b.BF16, 4096, 1536, 8960, 16, b.PATH_MATERIALISE)
    b.isopo_set_store_format(b.STORE_E4M3_SPLIT)                      # the same two bytes per element
    try:
        assert b.isopo_workspace_bytes(b.BF16, 4096, 1536, 8960, 16, b.PATH_MATERIALISE) == base
    finally:
        b.isopo_set_store_format(b.STORE_BF16)
    b.isopo_set_deterministic(True)                                   # per-CTA partial sums of K live in the workspace
    try:
        assert b.isopo_workspace_bytes(b.BF16, 4096, 1536, 8960, 16, b.PATH_MATERIALISE) >= base + 160 * 16 * 16 * 4
        assert b.isopo_workspace_bytes(b.BF16, 4096, 1536, 8960, 16, b.PATH_GRAM) == \
            b.isopo_workspace_bytes(b.BF16, 4096, 1536, 8960, 16, b.PATH_GRAM)
    finally:
        b.isopo_set_deterministic(False)
    assert b.isopo_workspace_bytes(b.BF16, 4096, 1536, 8960, 16, b.PATH_MATERIALISE) == base
    assert not b.isopo_debug_build()
    # interacting solve for more than 256 sequences: lower block triangle of 32 x 32 float32 blocks in the workspace
    assert b.isopo_transform_large_workspace_bytes(1024) == 528 * 4096
    assert b.isopo_transform_large_workspace_bytes(257) == 45 * 4096
    assert b.isopo_transform_large_workspace_bytes(0) == 0 and b.isopo_transform_large_workspace_bytes(1025) == 0
    large = lambda **kw: b.lib.isopo_transform_advantages_large(  # noqa: E731
        fake, fake, kw.get("B", 300), kw.get("lam", 0.1), fake, kw.get("ws", fake), kw.get("n", 1 << 22), fake, None)
    assert large(B=0) == b.ERR_INVALID_ARG and large(lam=-1.0) == b.ERR_INVALID_ARG
    assert large(ws=None) == b.ERR_INVALID_ARG and large(ws=fake + 4) == b.ERR_INVALID_ARG
    assert large(B=1025) == b.ERR_UNSUPPORTED
    assert large(n=55 * 4096 - 1) == b.ERR_WORKSPACE                    # 300 sequences: 10 block rows, 55 blocks


def test_binding_has_no_fallback():
    src = open(os.path.join(ROOT, "paper_2512_23353_b200", "binding.py")).read()
    assert "oracle" not in src.replace("CPU oracle", "")
    assert "ImportError" in src
