"""kvq_decode_static: the decode entry point that allocates no device memory.

Collected last on purpose (the file name sorts after every other test file), so a run that stops at the
first failure has already been through the rest of the suite.

Who needs it: an embedder that owns all of HBM through its own pool, or that cannot afford an allocation
(and the device-wide synchronisation it brings) once its decode loop runs.  kvq_decode allocates a status
word and the tensor-core kernel's table on a plan's first use; this variant keeps both in a fixed block
inside the library, shared by all calls.  The test checks it against kvq_decode through the C ABI on calls
in a row, including a change of plan between calls (the shared table must then be rewritten), and that a
plan too large for the block is refused on the host.
"""
import numpy as np
import pytest
import torch

from paper_2605_05699_b200 import binding as kb
from paper_2605_05699_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

G = wl.GROUP


def _compressed(plan, N, seed, n_lambda, rpl):
    x = wl.make_vectors(N, plan.D, "f16", "k_outlier", seed, device="cuda")
    lam = wl.make_lambda(n_lambda, plan.D, seed + 1, device="cuda")
    packed, scales = plan.empty_packed(N), plan.empty_scales(N)
    kb.kvq_encode(plan.handle, x, lam, packed, scales, rpl)
    return packed, scales, lam


def test_static_decode_matches_kvq_decode_on_calls_in_a_row():
    D = 128
    plans = [kb.Plan(D, G, 11), kb.Plan(D, G, 12)]
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    # plan A, plan A again (table reused), plan B (table rewritten), plan A (rewritten back)
    for call, (pi, N, n_lambda, rpl) in enumerate([(0, 5000, 1, 0), (0, 777, 3, 300), (1, 5000, 2, 2500), (0, 129, 1, 0)]):
        plan = plans[pi]
        packed, scales, lam = _compressed(plan, N, 100 + call, n_lambda, rpl)
        want = torch.empty(N, D, dtype=torch.float16, device="cuda")
        kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_FFT, kb.KVQ_IMPL_GEMM)
        kb.kvq_decode(plan.handle, packed, scales, lam, want, rpl)
        got = torch.full((N + 1, D), -3.0, dtype=torch.float16, device="cuda")
        kb.kvq_decode_static(plan.handle, packed, scales, lam, got[:N], rpl, status_word=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0, "a device-side wait timed out"
        assert bool((got[N] == -3.0).all()), "wrote past the last row"
        g, w = got[:N].float().cpu().numpy().astype(np.float64), want.float().cpu().numpy().astype(np.float64)
        rel = parity.rel_l2_rows(g, w)
        assert rel.max() <= parity.REL_L2, "call %d: relative L2 %.3g against kvq_decode" % (call, rel.max())
    # without a caller-owned status word the flag stays inside the block; the result is the same
    plan = plans[1]
    packed, scales, lam = _compressed(plan, 1000, 300, 1, 0)
    a = torch.empty(1000, D, dtype=torch.float16, device="cuda")
    b = torch.empty_like(a)
    kb.kvq_decode_static(plan.handle, packed, scales, lam, a)
    kb.kvq_decode_static(plan.handle, packed, scales, lam, b)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    for p in plans:
        p.close()


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
    p.close()
