"""The C ABI from plain C: tests/c_client.c includes only include/wht_affine.h and the CUDA runtime's C
header, is compiled as C99 and linked against the in-tree library.  Without a GPU: it compiles, links, and
its argument-error path runs.  With one: it runs the forward and the backward on a seeded problem and its
output file is compared with the oracle (Eq. 1 and its chain rule)."""
import os
import subprocess
import sys

import numpy as np
import pytest

import oracle
from helpers import assert_grad_vec, assert_rows_fp32
from paper_2603_08343_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


@pytest.fixture(scope="module")
def client(tmp_path_factory):
    from paper_2603_08343_b200 import build
    lib = build.build()
    libdir = os.path.dirname(lib)
    exe = str(tmp_path_factory.mktemp("c_client") / "c_client")
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
           "-isystem", os.path.join(CUDA, "include"), os.path.join(ROOT, "tests", "c_client.c"), "-o", exe,
           "-L", libdir, "-lwht_affine", "-L", os.path.join(CUDA, "lib64"), "-lcudart",
           f"-Wl,-rpath,{libdir}", f"-Wl,-rpath,{os.path.join(CUDA, 'lib64')}"]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    assert proc.returncode == 0, proc.stdout + proc.stderr
    return exe


def test_the_header_is_valid_c99_and_a_c_program_links(client):
    assert subprocess.run([client]).returncode == 0  # the argument-error path: no GPU needed


@pytest.mark.gpu
def test_a_c_program_gets_the_oracles_values(client, tmp_path):
    T, d = 301, 1024
    w = wl.Workload("cclient", T, d, wl.WHT_F32, "normal", 5100, True, "")
    x, dy = wl.gen_full(w, "x").numpy(), wl.gen_full(w, "dy").numpy()
    a, b = (t.numpy() for t in wl.gen_params(w))
    fin, fout = str(tmp_path / "in.bin"), str(tmp_path / "out.bin")
    np.concatenate([x.ravel(), dy.ravel(), a, b]).astype("<f4").tofile(fin)
    proc = subprocess.run([client, str(T), str(d), fin, fout], capture_output=True, text=True)
    assert proc.returncode == 0, proc.stderr
    out = np.fromfile(fout, dtype="<f4").astype(np.float64)
    n = T * d
    y, dx, da, db = out[:n].reshape(T, d), out[n:2 * n].reshape(T, d), out[2 * n:2 * n + d], out[2 * n + d:]
    x64, dy64, a64, b64 = (v.astype(np.float64) for v in (x, dy, a, b))
    assert_rows_fp32(y, oracle.wht_affine_fwd(x64, a64, b64), x64, "C client y")
    ref_dx, ref_da, ref_db = oracle.wht_affine_bwd(dy64, x64, a64)
    assert_rows_fp32(dx, ref_dx, a64[None, :] * dy64, "C client dx")
    assert_grad_vec(da, ref_da, "C client da")
    assert_grad_vec(db, ref_db, "C client db")
