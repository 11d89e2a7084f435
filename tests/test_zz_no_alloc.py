"""kvq_decode_static: the decode entry point that allocates no device memory.

Collected last on purpose (the file name sorts after every other test file), so a run that stops at the
first failure has already been through the rest of the suite.

Who needs it: an embedder that owns all of HBM through its own pool, or that cannot afford an allocation
(and the device-wide synchronisation it brings) once its decode loop runs.  kvq_decode allocates a status
word and the tensor-core kernel's table on a plan's first use; this variant keeps both in a fixed block
inside the library, shared by all calls.  The tests hold it to the fp64 oracle and to kvq_decode through the
C ABI on calls in a row, including a change of plan between calls (the shared table must then be rewritten),
read the driver's free-memory figure around calls on plans that were never used anywhere else, replay a
captured call after another plan has used the block, and check the host-side refusals.
"""
import numpy as np
import pytest
import torch

from oracle import kvq_oracle as ko
from paper_2605_05699_b200 import binding as kb
from paper_2605_05699_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

G = wl.GROUP
D = 128


def _compressed(seed_plan, N, seed, n_lambda, rpl):
    """Codes, scales and lambda for N vectors, made with a helper plan of the same seed (same sign diagonal), so that
    the plan handed to kvq_decode_static has never been near kvq_encode or kvq_decode."""
    helper = kb.Plan(D, G, seed_plan)
    x = wl.make_vectors(N, D, "f16", "k_outlier", seed, device="cuda")
    lam = wl.make_lambda(n_lambda, D, seed + 1, device="cuda")
    packed, scales = helper.empty_packed(N), helper.empty_scales(N)
    kb.kvq_encode(helper.handle, x, lam, packed, scales, rpl)
    want = torch.empty(N, D, dtype=torch.float16, device="cuda")
    kb.kvq_plan_set_impl(helper.handle, kb.KVQ_IMPL_AUTO, kb.KVQ_IMPL_GEMM)
    kb.kvq_decode(helper.handle, packed, scales, lam, want, rpl)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(helper.handle) == 0
    helper.close()
    return packed, scales, lam, want


def _oracle_check(plan_seed, packed, scales, lam, got, rpl, label):
    sg = ko.signs(D, plan_seed)
    pk, sb = packed.cpu().numpy(), wl.raw_bits(scales)
    ob, o64 = ko.decode(pk, sb, sg, lam.cpu().numpy(), G, ko.F16, rpl, want_f64=True)
    return parity.check_decode(wl.raw_bits(got), ob, o64, ko.F16, label)


def test_static_decode_matches_the_oracle_and_kvq_decode_on_calls_in_a_row():
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    # plan A, plan A again (table reused), plan B (table rewritten), plan A (rewritten back)
    for call, (seed_plan, N, n_lambda, rpl) in enumerate([(11, 5000, 1, 0), (11, 777, 3, 300), (12, 5000, 2, 2500), (11, 129, 1, 0)]):
        packed, scales, lam, want = _compressed(seed_plan, N, 100 + call, n_lambda, rpl)
        plan = kb.Plan(D, G, seed_plan)           # a fresh plan: kvq_decode_static is the only call it ever sees
        got = torch.full((N + 1, D), -3.0, dtype=torch.float16, device="cuda")
        kb.kvq_decode_static(plan.handle, packed, scales, lam, got[:N], rpl, status_word=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0, "a device-side wait timed out"
        assert bool((got[N] == -3.0).all()), "wrote past the last row"
        _oracle_check(seed_plan, packed, scales, lam, got[:N], rpl, "static decode, call %d" % call)
        g, w = got[:N].float().cpu().numpy().astype(np.float64), want.float().cpu().numpy().astype(np.float64)
        rel = parity.rel_l2_rows(g, w)
        assert rel.max() <= parity.REL_L2, "call %d: relative L2 %.3g against kvq_decode" % (call, rel.max())
        assert plan.describe()[1] == 0, "the plan was given device tables"
        plan.close()
    # without a caller-owned status word the flag stays inside the block; the result is the same
    packed, scales, lam, _ = _compressed(12, 1000, 300, 1, 0)
    plan = kb.Plan(D, G, 12)
    a = torch.empty(1000, D, dtype=torch.float16, device="cuda")
    b = torch.empty_like(a)
    kb.kvq_decode_static(plan.handle, packed, scales, lam, a)
    kb.kvq_decode_static(plan.handle, packed, scales, lam, b)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    plan.close()


def test_static_decode_leaves_the_free_memory_figure_alone():
    """The driver's free-memory figure before and after calls on plans that nothing else has used.  The first call of a
    process loads the kernels' code (the CUDA runtime does that lazily and it shows in the figure), so one warm call comes
    first; from then on a new plan, another plan's table and a large call must not move it."""
    cases = [_compressed(21, 4000, 400, 1, 0), _compressed(22, 70000, 410, 4, 20000), _compressed(21, 300, 420, 1, 0)]
    outs = [torch.empty(c[0].shape[0], D, dtype=torch.float16, device="cuda") for c in cases]
    warm = kb.Plan(D, G, 20)
    kb.kvq_decode_static(warm.handle, cases[0][0], cases[0][1], cases[0][2], outs[0])
    torch.cuda.synchronize()
    warm.close()
    plans = [kb.Plan(D, G, s) for s in (21, 22, 21)]          # host objects only
    free0, _ = torch.cuda.mem_get_info()
    for plan, (packed, scales, lam, _), out, rpl in zip(plans, cases, outs, (0, 20000, 0)):
        kb.kvq_decode_static(plan.handle, packed, scales, lam, out, rpl)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, "device memory moved by %d bytes across kvq_decode_static calls" % (free0 - free1)
    for plan, seed_plan, (packed, scales, lam, _), out, rpl in zip(plans, (21, 22, 21), cases, outs, (0, 20000, 0)):
        assert plan.describe()[1] == 0
        _oracle_check(seed_plan, packed, scales, lam, out, rpl, "static decode, fresh plan %d" % seed_plan)
        plan.close()


def test_a_captured_static_decode_brings_its_own_table():
    """A call recorded into a CUDA graph is replayed after another plan has rewritten the shared block: the recording holds
    the table fill, so the replay decodes with its own plan's signs whatever ran in between."""
    pa, sa, la, _ = _compressed(31, 3000, 500, 1, 0)
    pb, sb_, lb, _ = _compressed(32, 3000, 510, 1, 0)
    plan_a, plan_b = kb.Plan(D, G, 31), kb.Plan(D, G, 32)
    out_a = torch.zeros(3000, D, dtype=torch.float16, device="cuda")
    out_b = torch.zeros(3000, D, dtype=torch.float16, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):                 # the block's address is looked up on the first call: before any capture
        kb.kvq_decode_static(plan_a.handle, pa, sa, la, out_a)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):                 # recorded while plan A's table is the cached one
        kb.kvq_decode_static(plan_a.handle, pa, sa, la, out_a)
    for rep in range(2):
        out_a.zero_()
        kb.kvq_decode_static(plan_b.handle, pb, sb_, lb, out_b)     # plan B takes the block over ...
        graph.replay()                                               # ... and the replay must not decode with B's signs
        kb.kvq_decode_static(plan_b.handle, pb, sb_, lb, out_b)     # an eager call after a replay: the host's note about
        torch.cuda.synchronize()                                     # the block must not have been fooled either
        _oracle_check(31, pa, sa, la, out_a, 0, "replayed static decode, round %d" % rep)
        _oracle_check(32, pb, sb_, lb, out_b, 0, "eager static decode after a replay, round %d" % rep)
    plan_a.close()
    plan_b.close()


def test_static_decode_of_a_lambda_row_no_fp16_operand_can_carry():
    """An entry at the 1e-6 clamp (Sec. 5.1 item 1) beside ordinary ones: the kernel redoes such a row's tiles in fp32 inside
    the same launch, with the table in the fixed block, and still allocates nothing."""
    N, rpl = 3000, 1000
    helper = kb.Plan(D, G, 41)
    x = wl.make_vectors(N, D, "f16", "k_outlier", 600, device="cuda")
    lam = wl.make_lambda(3, D, 601, device="cuda")
    lam[1, 9] = 1e-6
    packed, scales = helper.empty_packed(N), helper.empty_scales(N)
    kb.kvq_encode(helper.handle, x, lam, packed, scales, rpl)
    torch.cuda.synchronize()
    helper.close()
    plan = kb.Plan(D, G, 41)
    got = torch.empty(N, D, dtype=torch.float16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kb.kvq_decode_static(plan.handle, packed, scales, lam, got, rpl, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    sg = ko.signs(D, 41)
    ob, o64 = ko.decode(packed.cpu().numpy(), wl.raw_bits(scales), sg, lam.cpu().numpy(), G, ko.F16, rpl, want_f64=True)
    ok = np.abs(o64).max(axis=1) < 0.25 * 65504.0
    assert ok[:rpl].all() and ok[2 * rpl:].all() and ok[rpl:2 * rpl].mean() > 0.3
    parity.check_decode(wl.raw_bits(got)[ok], ob[ok], o64[ok], ko.F16, "static decode, wide lambda row")
    assert plan.describe()[1] == 0
    plan.close()


def test_static_decode_refuses_what_does_not_fit():
    lam256 = torch.ones(256, device="cuda")
    big = kb.Plan(256, G, 1)
    out = torch.empty(8, 256, dtype=torch.float16, device="cuda")
    with pytest.raises(kb.KvqError) as e:
        kb.kvq_decode_static(big.handle, big.empty_packed(8), big.empty_scales(8), lam256, out)
    assert e.value.status == kb.KVQ_ERR_SCRATCH_LIMIT
    big.close()
    small = kb.Plan(96, G, 1)
    out = torch.empty(8, 96, dtype=torch.float16, device="cuda")
    with pytest.raises(kb.KvqError) as e:
        kb.kvq_decode_static(small.handle, small.empty_packed(8), small.empty_scales(8), torch.ones(96, device="cuda"), out)
    assert e.value.status == kb.KVQ_ERR_UNSUPPORTED_DIM
    small.close()
    p = kb.Plan(128, G, 1)
    out = torch.empty(8, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(kb.KvqError) as e:
        kb.kvq_decode_static(p.handle, p.empty_packed(8), p.empty_scales(8), torch.ones(128, device="cuda"), out)
    assert e.value.status == kb.KVQ_ERR_UNSUPPORTED_DIM
    # 2^31 rows and more are refused on the host, before anything is enqueued (the pointers are never read)
    n0 = kb.kvq_launch_count()
    st = kb.lib().kvq_decode_static(p.handle, 4096, 4096, 1 << 31, torch.ones(128, device="cuda").data_ptr(), 1, 0, 4096, kb.KVQ_F16, None, None)
    assert st == kb.KVQ_ERR_INVALID_ARG and kb.kvq_launch_count() == n0
    p.close()
