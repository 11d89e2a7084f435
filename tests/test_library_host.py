"""Host-side checks of libkvq that need no GPU: the library loads, exports every symbol the header
declares, builds plans, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

from oracle import kvq_oracle as ko
from paper_2605_05699_b200 import binding as kb
from paper_2605_05699_b200 import build as kbuild
from paper_2605_05699_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built_library():
    kbuild.build()


def test_library_exports_every_symbol_the_header_declares():
    text = open(os.path.join(ROOT, "include", "kvq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(kvq_[a-z_0-9]+)\s*\(", text))
    assert declared == set(kb.EXPORTS)
    L = ctypes.CDLL(kb.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), name


@pytest.mark.parametrize("D", [64, 96, 128, 160, 256])
def test_plan_signs_match_the_oracles_independent_generator(D):
    for seed in (0, 1, 1234567, 2**63 + 5):
        p = kb.Plan(D, 32, seed)
        assert np.array_equal(p.signs(), ko.signs(D, seed))
        p.close()


def test_plan_describe_reports_the_mixed_radix_factorisation():
    want = {64: [4, 4, 2], 96: [4, 4, 3], 128: [4, 4, 4], 160: [4, 4, 5], 256: [4, 4, 4, 2]}
    for D, radices in want.items():
        p = kb.Plan(D, 32, 1)
        r, table_bytes = kb.kvq_plan_describe(p.handle)
        assert r == radices and int(np.prod(r)) == D // 2
        assert table_bytes == 0  # no device tables before the first GPU call
        p.close()


def test_unsupported_dims_and_groups_are_rejected():
    L = kb.lib()
    h = ctypes.c_void_p()
    for D, g in [(100, 32), (127, 32), (0, 32), (512, 32), (128, 16), (128, 0), (96, 64)]:
        assert L.kvq_plan_create(D, g, 1, ctypes.byref(h)) == kb.KVQ_ERR_UNSUPPORTED_DIM
        assert h.value is None
    assert L.kvq_plan_create(128, 32, 1, None) == kb.KVQ_ERR_INVALID_ARG
    # base variants: one scale per vector (group = D) and 8-bit codes are plans too; nothing else is
    for D, g, b in [(128, 128, 4), (96, 96, 8), (256, 32, 8), (64, 64, 8)]:
        p = kb.Plan(D, g, 1, bits=b)
        assert p.empty_packed(3, "cpu").shape == (3, D * b // 8) and p.empty_scales(3, "cpu").shape == (3, D // g)
        p.close()
    for D, g, b in [(128, 32, 5), (128, 32, 16), (128, 32, 0), (128, 64, 8), (96, 128, 4)]:
        assert L.kvq_plan_create_ex(D, g, b, 1, ctypes.byref(h)) == kb.KVQ_ERR_UNSUPPORTED_DIM
        assert h.value is None


def test_the_header_is_plain_c():
    # the boundary is a C ABI: the header must compile as C, on its own
    import subprocess
    import tempfile

    hdr = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "kvq.h")
    with tempfile.TemporaryDirectory() as d:
        src = os.path.join(d, "use.c")
        with open(src, "w") as f:
            f.write('#include "%s"\nint main(void) { kvq_plan_t *p = 0; return (int)kvq_plan_destroy(p) + (int)KVQ_IMPL_MATVEC * 0; }\n' % hdr)
        r = subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-fsyntax-only", src], capture_output=True, text=True)
        assert r.returncode == 0, r.stderr


def test_rotation_is_validated_on_the_host():
    p = kb.Plan(128, 32, 1)
    R = wl.make_rotation(128, 3)
    assert torch.allclose(R @ R.T, torch.eye(128), atol=1e-5)
    p.set_rotation(R)            # before any GPU use: kept on the host until the tables are built
    p.set_rotation(None)
    bad = R.clone()
    bad[5, 7] = float("nan")
    with pytest.raises(kb.KvqError) as e:
        p.set_rotation(bad)
    assert e.value.status == kb.KVQ_ERR_INVALID_ARG
    with pytest.raises(ValueError):
        p.set_rotation(R[:64, :64])
    p.close()
    for q in (kb.Plan(128, 128, 1), kb.Plan(128, 32, 1, bits=8)):    # every layout takes a rotation
        q.set_rotation(R)
        q.close()
    near = wl.make_rotation(64, 4, near_identity=0.02)
    assert torch.allclose(near @ near.T, torch.eye(64), atol=1e-5) and float((near - torch.eye(64)).abs().max()) < 0.5


def test_prepare_and_wait_limit_check_their_arguments_before_cuda():
    L = kb.lib()
    p = kb.Plan(128, 32, 1)
    assert L.kvq_plan_prepare(None, kb.KVQ_F16) == kb.KVQ_ERR_INVALID_ARG
    assert L.kvq_plan_prepare(p.handle, 2) == kb.KVQ_ERR_INVALID_ARG           # dtype
    assert L.kvq_plan_set_wait_limit(None, 4) == kb.KVQ_ERR_INVALID_ARG
    assert L.kvq_plan_set_wait_limit(p.handle, 4) == kb.KVQ_OK
    assert L.kvq_plan_set_wait_limit(p.handle, 0) == kb.KVQ_OK
    if not torch.cuda.is_available():
        # valid arguments, no device: the failing CUDA call is reported, nothing is computed on the host
        assert L.kvq_plan_prepare(p.handle, kb.KVQ_F16) == kb.KVQ_ERR_CUDA
        assert kb.kvq_plan_describe(p.handle)[1] == 0
    p.close()


def test_bad_arguments_are_rejected_on_the_host():
    L = kb.lib()
    p = kb.Plan(128, 32, 1)
    A = 4096  # fake, 16-byte aligned "device" addresses: validation must fail before any is dereferenced
    enc = lambda *a: L.kvq_encode(*a)
    assert enc(None, A, 0, 8, A, 1, 0, A, A, None) == kb.KVQ_ERR_INVALID_ARG
    assert enc(p.handle, None, 0, 8, A, 1, 0, A, A, None) == kb.KVQ_ERR_INVALID_ARG
    assert enc(p.handle, A, 0, 8, None, 1, 0, A, A, None) == kb.KVQ_ERR_INVALID_ARG
    assert enc(p.handle, A, 0, 8, A, 1, 0, None, A, None) == kb.KVQ_ERR_INVALID_ARG
    assert enc(p.handle, A, 0, 8, A, 1, 0, A, None, None) == kb.KVQ_ERR_INVALID_ARG
    assert enc(p.handle, A, 0, -1, A, 1, 0, A, A, None) == kb.KVQ_ERR_INVALID_ARG
    assert enc(p.handle, A, 7, 8, A, 1, 0, A, A, None) == kb.KVQ_ERR_INVALID_ARG       # dtype
    assert enc(p.handle, A, 0, 8, A, 0, 0, A, A, None) == kb.KVQ_ERR_INVALID_ARG       # n_lambda
    assert enc(p.handle, A, 0, 8, A, 2, 0, A, A, None) == kb.KVQ_ERR_INVALID_ARG       # rows_per_lambda
    assert enc(p.handle, A, 0, 9, A, 2, 4, A, A, None) == kb.KVQ_ERR_INVALID_ARG       # table too short
    assert enc(p.handle, A + 2, 0, 8, A, 1, 0, A, A, None) == kb.KVQ_ERR_ALIGNMENT
    assert enc(p.handle, A, 0, 8, A, 1, 0, A + 8, A, None) == kb.KVQ_ERR_ALIGNMENT
    assert enc(p.handle, A, 0, 8, A + 4, 1, 0, A, A, None) == kb.KVQ_ERR_ALIGNMENT
    assert enc(p.handle, A, 0, 0, A, 1, 0, A, A, None) == kb.KVQ_OK                    # N == 0: no-op
    dec = lambda *a: L.kvq_decode(*a)
    assert dec(p.handle, None, A, 8, A, 1, 0, A, 0, None) == kb.KVQ_ERR_INVALID_ARG
    assert dec(p.handle, A, A, 8, A, 1, 0, None, 0, None) == kb.KVQ_ERR_INVALID_ARG
    assert dec(p.handle, A, A, 8, A, 1, 0, A + 1, 0, None) == kb.KVQ_ERR_ALIGNMENT
    assert dec(p.handle, A, A, 0, A, 1, 0, A, 1, None) == kb.KVQ_OK
    app = lambda *a: L.kvq_append(*a)
    assert app(p.handle, A, 0, 4, A, 1, 0, A, A, 16, 16, None) == kb.KVQ_ERR_INVALID_ARG  # pos == T_max
    assert app(p.handle, A, 0, 4, A, 1, 0, A, A, 16, -1, None) == kb.KVQ_ERR_INVALID_ARG
    assert app(p.handle, A, 0, 4, A, 1, 0, A, A, 0, 0, None) == kb.KVQ_ERR_INVALID_ARG
    assert app(p.handle, A, 0, 0, A, 1, 0, A, A, 16, 3, None) == kb.KVQ_OK
    # the position-in-device-memory forms: the word itself is checked for presence and alignment, its value on the device
    app_at = lambda *a: L.kvq_append_at(*a)
    assert app_at(p.handle, A, 0, 4, A, 1, 0, A, A, 16, None, None) == kb.KVQ_ERR_INVALID_ARG
    assert app_at(p.handle, A, 0, 4, A, 1, 0, A, A, 16, A + 4, None) == kb.KVQ_ERR_ALIGNMENT
    assert app_at(p.handle, A, 0, 4, A, 1, 0, A, A, 0, A, None) == kb.KVQ_ERR_INVALID_ARG     # T_max
    assert app_at(None, A, 0, 4, A, 1, 0, A, A, 16, A, None) == kb.KVQ_ERR_INVALID_ARG
    assert app_at(p.handle, None, 0, 4, A, 1, 0, A, A, 16, A, None) == kb.KVQ_ERR_INVALID_ARG
    assert app_at(p.handle, A, 0, 0, A, 1, 0, A, A, 16, A, None) == kb.KVQ_OK
    fl_at = lambda *a: L.kvq_flush_block_at(*a)
    assert fl_at(p.handle, A, 0, 4, 8, A, 1, 0, A, A, A, 16, None, None) == kb.KVQ_ERR_INVALID_ARG
    assert fl_at(p.handle, A, 0, 4, 8, A, 1, 0, A, A, A, 16, A + 4, None) == kb.KVQ_ERR_ALIGNMENT
    assert fl_at(p.handle, A, 0, 4, 17, A, 1, 0, A, A, A, 16, A, None) == kb.KVQ_ERR_INVALID_ARG  # more rows than the cache has
    assert fl_at(p.handle, A, 0, 4, 8, A, 1, 0, A, A, None, 16, A, None) == kb.KVQ_ERR_INVALID_ARG
    assert fl_at(p.handle, A, 0, 4, 0, A, 1, 0, A, A, A, 16, A, None) == kb.KVQ_OK
    assert L.kvq_plan_set_impl(p.handle, 9, 0) == kb.KVQ_ERR_INVALID_ARG
    assert L.kvq_plan_get_signs(p.handle, None) == kb.KVQ_ERR_INVALID_ARG
    assert kb.kvq_plan_device_status(p.handle) == 0
    p.close()
    assert L.kvq_plan_destroy(None) == kb.KVQ_OK


def test_status_strings_and_launch_counter():
    names = [kb.status_string(i) for i in range(7)]
    assert names[0] == "KVQ_OK" and len(set(names)) == 7 and all(n.startswith("KVQ_") for n in names)
    assert kb.kvq_launch_count() >= 0


def test_compute_without_a_device_fails_loudly_never_silently():
    import torch

    if torch.cuda.is_available():
        pytest.skip("a device is present")
    L = kb.lib()
    p = kb.Plan(128, 32, 1)
    A = 4096
    assert L.kvq_encode(p.handle, A, 0, 8, A, 1, 0, A, A, None) == kb.KVQ_ERR_CUDA
    assert L.kvq_decode(p.handle, A, A, 8, A, 1, 0, A, 0, None) == kb.KVQ_ERR_CUDA
    p.close()
