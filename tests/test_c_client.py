"""The boundary is a C library: `include/isopo.h` compiles as plain C99, and a caller written in C (no Python, no
PyTorch: `tests/c_client/isopo_client.c`, device memory from the CUDA runtime) gets the oracle's K, coefficients and
dW out of the three calls."""

import os
import struct
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PKG = os.path.join(ROOT, "paper_2512_23353_b200")
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")
SRC = os.path.join(ROOT, "tests", "c_client", "isopo_client.c")


def _compile(tmp_path):
    from paper_2512_23353_b200 import build
    build.build()
    exe = str(tmp_path / "isopo_client")
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-O1", SRC, "-o", exe,
           "-I", os.path.join(ROOT, "include"), "-isystem", os.path.join(CUDA, "include"),
           "-L", PKG, "-lisopo", "-L", os.path.join(CUDA, "lib64"), "-lcudart",
           "-Wl,-rpath," + PKG, "-Wl,-rpath," + os.path.join(CUDA, "lib64")]
    r = subprocess.run(cmd, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    return exe


def test_header_is_plain_c(tmp_path):
    src = tmp_path / "only_header.c"
    src.write_text('#include "isopo.h"\nint main(void) { return (int)ISOPO_OK; }\n')
    r = subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only",
                        "-I", os.path.join(ROOT, "include"), str(src)], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr


def test_c_client_builds_and_links(tmp_path):
    """gcc, C99, warnings as errors; links against libisopo.so and the CUDA runtime only."""
    exe = _compile(tmp_path)
    r = subprocess.run([exe], capture_output=True, text=True)       # no arguments: usage, exit code 1, no CUDA call
    assert r.returncode == 1 and "usage" in r.stderr


@pytest.mark.gpu
@pytest.mark.parametrize("path", [1, 2])        # ISOPO_PATH_GRAM, ISOPO_PATH_MATERIALISE
def test_c_client_matches_oracle(tmp_path, path):
    from oracle import isopo_oracle as orc
    from paper_2512_23353_b200 import workloads as wl
    from tests._util import rel_fro

    exe = _compile(tmp_path)
    w = wl.WORKLOADS["tiny_f32"]                 # the float32 configuration: 64 -> 64, 8 sequences of 16..64 tokens
    off, A = wl.microbatch(w)
    T, B = int(off[-1]), len(A)
    layer = w.layers[0]
    X, dY = wl.layer_inputs_host(w, layer, T)
    G = orc.sequence_gradients(X, dY, off)
    K_o = orc.ntk(G)
    lam = float(np.float32(1e-3 * np.mean(np.diag(K_o))))
    c_o = orc.transform_advantages(K_o, A.astype(np.float64), orc.INTERACTING, lam)
    dW_o = orc.weight_gradient(G, c_o)
    problem, result = tmp_path / "problem.bin", tmp_path / "result.bin"
    with open(problem, "wb") as f:
        f.write(struct.pack("<5q", T, layer.d_in, layer.d_out, B, path))
        f.write(struct.pack("<d", lam))
        f.write(np.asarray(off, dtype="<i8").tobytes())
        for a in (X, dY, A):
            f.write(np.ascontiguousarray(a, dtype="<f4").tobytes())
    r = subprocess.run([exe, str(problem), str(result)], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    raw = open(result, "rb").read()
    info = struct.unpack_from("<i", raw, 0)[0]
    vals = np.frombuffer(raw, dtype="<f4", offset=4)
    K, c, dW = vals[:B * B].reshape(B, B), vals[B * B:B * B + B], vals[B * B + B:].reshape(layer.d_out, layer.d_in)
    assert info == 0
    errs = (rel_fro(K, K_o), rel_fro(c, c_o), rel_fro(dW, dW_o))
    print(f"[parity] C client, path {path}: K={errs[0]:.3e}, c={errs[1]:.3e}, dW={errs[2]:.3e}")
    assert max(errs) <= 1e-5
