"""The range-checking build (libisopo_debug.so, -DISOPO_DEBUG) compares every data-dependent index of the
kernels with its buffer's extent before the access and reports a violation as ISOPO_INFO_BOUNDS in
*info.  Here the parity tests with the most awkward addressing (ragged tails of every residue, widths
off the tile grid, single-token sequences, every stored-piece box shape, segments cut by token
chunks, sample rows that fill part of a tile) run again on that build in a child process: they all
assert info == 0, so passing means no index left its buffer, and the results still match the oracle."""

import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_edge_shape_parity_on_the_range_checking_build():
    from paper_2512_23353_b200 import build as _build

    path = _build.build(debug=True)
    assert os.path.exists(path)
    env = dict(os.environ, ISOPO_LIB_VARIANT="debug")
    probe = subprocess.run([sys.executable, "-c",
                            "from paper_2512_23353_b200 import binding as b; assert b.isopo_debug_build(); print(b.LIB_PATH)"],
                           cwd=ROOT, env=env, capture_output=True, text=True)
    assert probe.returncode == 0 and "libisopo_debug.so" in probe.stdout, probe.stderr
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu",
                        "tests/test_parity_bf16.py", "tests/test_parity_f32.py", "tests/test_weight_grad_fold_gpu.py",
                        "tests/test_sampled_gpu.py", "tests/test_gram_shared_gpu.py", "tests/test_workspace_tag_gpu.py",
                        "tests/test_shared_x_stored_gpu.py", "tests/test_split_store_gpu.py",
                        "-k", "not small_llm_config"],
                       cwd=ROOT, env=env, capture_output=True, text=True)
    tail = "\n".join(r.stdout.splitlines()[-15:])
    print(tail)
    assert r.returncode == 0, tail + r.stderr[-2000:]


def test_the_default_library_is_not_the_debug_build():
    from paper_2512_23353_b200 import binding as b
    if os.environ.get("ISOPO_LIB_VARIANT") != "debug":
        assert not b.isopo_debug_build()
