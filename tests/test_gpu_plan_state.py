"""The plan's device state: explicit preparation (after which compute calls can be captured without a warm call) and
the reporting of a bounded device-side wait that ran out."""
import numpy as np
import pytest
import torch

from oracle import kvq_oracle as ko
from paper_2605_05699_b200 import binding as kb
from paper_2605_05699_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

G = wl.GROUP
DT = {"f16": ko.F16, "bf16": ko.BF16}


@pytest.mark.parametrize("D,dtype,N", [(128, "f16", 6000), (256, "bf16", 3000), (96, "f16", 700)])
def test_prepared_plan_is_captured_without_a_warm_call(D, dtype, N):
    """A stream capture refuses allocations and blocking copies.  After kvq_plan_prepare the very first encode, append and
    decode of a plan are recorded into a CUDA graph as they are; the replay must give what the oracle gives."""
    tdt = wl.torch_dtype(dtype)
    plan = kb.Plan(D, G, 400 + D)
    sg = plan.signs()
    x = wl.make_vectors(N, D, dtype, "k_outlier", 401)
    lam = wl.make_lambda(2, D, 402)
    rpl = (N + 1) // 2
    xd, lamd = x.cuda(), lam.cuda()
    packed, scales = plan.empty_packed(N).zero_(), plan.empty_scales(N).zero_()
    out = torch.zeros(N, D, dtype=tdt, device="cuda")
    cache_p = torch.zeros(4, 3, D // 2, dtype=torch.uint8, device="cuda")
    cache_s = torch.zeros(4, 3, D // G, dtype=torch.float16, device="cuda")
    assert plan.describe()[1] == 0
    kb.kvq_plan_prepare(plan.handle, tdt)
    assert plan.describe()[1] > 0                      # the tables exist now
    kb.kvq_plan_prepare(plan.handle, tdt)              # idempotent
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        kb.kvq_encode(plan.handle, xd, lamd, packed, scales, rpl)
        kb.kvq_append(plan.handle, xd[:4], lamd, cache_p, cache_s, 1, 2)
        kb.kvq_decode(plan.handle, packed, scales, lamd, out, rpl)
    graph.replay()
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    ora = ko.encode(wl.raw_bits(x), DT[dtype], sg, lam.numpy(), G, rpl, want_v=True)
    pk, sb = packed.cpu().numpy(), wl.raw_bits(scales)
    parity.check_encode(pk, sb, ora, G, "captured encode", min_agree=0.9995 if N * D < 500000 else parity.CODE_AGREEMENT)
    ob, o64 = ko.decode(pk, sb, sg, lam.numpy(), G, DT[dtype], rpl, want_f64=True)
    parity.check_decode(wl.raw_bits(out), ob, o64, DT[dtype], "captured decode")
    assert bool((cache_p[:, 1] != 0).any()) and not bool(cache_p[:, [0, 2]].any())
    plan.close()


def test_prepare_checks_its_arguments_first():
    L = kb.lib()
    p = kb.Plan(128, G, 1)
    assert L.kvq_plan_prepare(None, kb.KVQ_F16) == kb.KVQ_ERR_INVALID_ARG
    assert L.kvq_plan_prepare(p.handle, 5) == kb.KVQ_ERR_INVALID_ARG
    assert p.describe()[1] == 0
    p.close()


def test_a_bounded_wait_that_runs_out_is_reported_and_service_returns():
    """Every wait inside the kernels is bounded and ends in a status bit, never in a hang.  With the host-settable limit of
    the tensor-core encode kernel's first wait cut to one poll, a one-tile call gives up at a point where the waiting role
    has nothing in flight: the call returns, writes nothing, the status word carries the slot-time-out bit and reads as
    KVQ_ERR_TIMEOUT; after clearing it and restoring the limit the same call is correct."""
    D, N = 128, 100                                   # one tile
    plan = kb.Plan(D, G, 500)
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_GEMM, kb.KVQ_IMPL_AUTO)
    sg = plan.signs()
    x = wl.make_vectors(N, D, "f16", "gaussian", 501)
    lam = wl.make_lambda(1, D, 502)
    xd, lamd = x.cuda(), lam.cuda()
    packed = torch.full((N, D // 2), 0xAB, dtype=torch.uint8, device="cuda")
    scales = torch.full((N, D // G), 1.25, dtype=torch.float16, device="cuda")
    kb.kvq_plan_set_wait_limit(plan.handle, 1)
    kb.kvq_encode(plan.handle, xd, lamd, packed, scales)
    torch.cuda.synchronize()                          # the launch ends by itself
    word = kb.kvq_plan_device_status(plan.handle)
    assert word & 7 == 4, "status word %d" % word     # bit 2: a wait for a pipeline slot ran out
    w = kb.ctypes.c_uint32()
    assert kb.lib().kvq_plan_device_status(plan.handle, kb.ctypes.byref(w)) == kb.KVQ_ERR_TIMEOUT
    assert bool((packed == 0xAB).all()) and bool((scales == 1.25).all())      # nothing was written
    kb.kvq_plan_clear_device_status(plan.handle)
    assert kb.kvq_plan_device_status(plan.handle) == 0
    kb.kvq_plan_set_wait_limit(plan.handle, 0)        # the default again
    kb.kvq_encode(plan.handle, xd, lamd, packed, scales)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    ora = ko.encode(wl.raw_bits(x), ko.F16, sg, lam.numpy(), G, want_v=True)
    parity.check_encode(packed.cpu().numpy(), wl.raw_bits(scales), ora, G, "encode after a reported time-out", min_agree=0.9995)
    plan.close()
