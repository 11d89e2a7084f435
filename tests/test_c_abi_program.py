"""The library used from plain C: tests/c_abi/roundtrip.c is compiled with gcc against include/kvq.h and libkvq.so,
allocates its own device buffers with the CUDA runtime and calls kvq_encode / kvq_decode; no Python object crosses the
boundary.  The files it writes are compared with the oracle."""
import os
import shutil
import subprocess

import numpy as np
import pytest
import torch

from oracle import kvq_oracle as ko
from paper_2605_05699_b200 import binding as kb
from paper_2605_05699_b200 import workloads as wl

from . import parity

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def build_program(tmp_path):
    if shutil.which("gcc") is None or not os.path.exists(os.path.join(CUDA, "include", "cuda_runtime_api.h")):
        pytest.skip("gcc or the CUDA runtime headers are not here")
    kb.lib()                                     # the library must exist (raises with the build hint otherwise)
    exe = str(tmp_path / "roundtrip")
    libdir = os.path.dirname(kb.LIB_PATH)
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-O1", os.path.join(ROOT, "tests", "c_abi", "roundtrip.c"),
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(CUDA, "include"), "-L", libdir, "-lkvq",
           "-L", os.path.join(CUDA, "lib64"), "-lcudart", "-Wl,-rpath," + libdir, "-Wl,-rpath," + os.path.join(CUDA, "lib64"), "-o", exe]
    r = subprocess.run(cmd, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    return exe


def write_inputs(tmp_path, D, N, dtype, n_lambda, seed):
    x = wl.make_vectors(N, D, dtype, "k_outlier", seed)
    lam = wl.make_lambda(n_lambda, D, seed + 1)
    wl.raw_bits(x).tofile(str(tmp_path / "x.bin"))
    lam.numpy().astype(np.float32).tofile(str(tmp_path / "lambda.bin"))
    return x, lam


def test_c_program_links_and_fails_loudly_without_a_device(tmp_path):
    exe = build_program(tmp_path)
    if torch.cuda.is_available():
        pytest.skip("a device is present: the GPU test runs the program")
    write_inputs(tmp_path, 128, 8, "f16", 1, 5)
    r = subprocess.run([exe, "128", "8", "0", "1", "0", "7", str(tmp_path)], capture_output=True, text=True)
    assert r.returncode == 1 and "->" in r.stderr          # a CUDA or library call reported its failure; nothing was computed
    assert not (tmp_path / "packed.bin").exists()


@pytest.mark.gpu
@pytest.mark.parametrize("D,N,dtype,n_lambda,rpl", [(128, 5000, "f16", 3, 1700), (256, 3001, "bf16", 1, 0), (96, 777, "f16", 1, 0)])
def test_c_program_round_trip_matches_the_oracle(tmp_path, D, N, dtype, n_lambda, rpl):
    exe = build_program(tmp_path)
    seed = 4242
    x, lam = write_inputs(tmp_path, D, N, dtype, n_lambda, 600 + D)
    r = subprocess.run([exe, str(D), str(N), "0" if dtype == "f16" else "1", str(n_lambda), str(rpl), str(seed), str(tmp_path)],
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout + r.stderr
    assert r.stdout.startswith("ok launches=2 status_word=0")
    G = wl.GROUP
    odt = ko.F16 if dtype == "f16" else ko.BF16
    sg = np.fromfile(str(tmp_path / "signs.bin"), dtype=np.int8)
    assert np.array_equal(sg, ko.signs(D, seed))
    pk = np.fromfile(str(tmp_path / "packed.bin"), dtype=np.uint8).reshape(N, D // 2)
    sb = np.fromfile(str(tmp_path / "scales.bin"), dtype=np.uint16).reshape(N, D // G)
    out = np.fromfile(str(tmp_path / "out.bin"), dtype=np.uint16).reshape(N, D)
    ora = ko.encode(wl.raw_bits(x), odt, sg, lam.numpy(), G, rpl, want_v=True)
    parity.check_encode(pk, sb, ora, G, "C caller encode")
    ob, o64 = ko.decode(pk, sb, sg, lam.numpy(), G, odt, rpl, want_f64=True)
    parity.check_decode(out, ob, o64, odt, "C caller decode")
