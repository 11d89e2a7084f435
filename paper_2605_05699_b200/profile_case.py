"""Runs one small, fixed case of one libkvq kernel a few times: the command to put under ncu.

    python -m paper_2605_05699_b200.profile_case --op decode --D 128 --dtype f16 --n 1048576 --impl auto --reps 3

The case is sized for a profiler capture: inputs and outputs larger than L2, well under a GB on the
device, a handful of launches, nothing else running.  It prints the CUDA-event time of the last launch
so the same command doubles as a quick timing probe (never quote a time taken under a profiler).
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as kb
from . import workloads as wl

IMPL = {"auto": kb.KVQ_IMPL_AUTO, "fft": kb.KVQ_IMPL_FFT, "gemm": kb.KVQ_IMPL_GEMM}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", choices=["encode", "decode", "append"], default="decode")
    ap.add_argument("--D", type=int, default=128)
    ap.add_argument("--dtype", choices=["f16", "bf16"], default="f16")
    ap.add_argument("--n", type=int, default=1 << 20)
    ap.add_argument("--impl", choices=list(IMPL), default="auto")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--kind", default="k_outlier")
    a = ap.parse_args()

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    D, G, N = a.D, wl.GROUP, a.n
    plan = kb.Plan(D, G, 3)
    x = wl.make_vectors(N, D, a.dtype, a.kind, 11, device=dev)
    lam = wl.make_lambda(1, D, 12, device=dev)
    packed, scales = plan.empty_packed(N), plan.empty_scales(N)
    out = torch.empty_like(x)
    # the compressed input of decode always comes from the fp32 FFT encoder
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_FFT, IMPL[a.impl])
    kb.kvq_encode(plan.handle, x, lam, packed, scales)
    kb.kvq_plan_set_impl(plan.handle, IMPL[a.impl], IMPL[a.impl])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(a.reps):
        e0.record()
        if a.op == "encode":
            kb.kvq_encode(plan.handle, x, lam, packed, scales)
        elif a.op == "decode":
            kb.kvq_decode(plan.handle, packed, scales, lam, out)
        else:
            kb.kvq_append(plan.handle, x[:4096], lam, packed.view(4096, -1, D // 2), scales.view(4096, -1, D // G), 1)
        e1.record()
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    assert kb.kvq_plan_device_status(plan.handle) == 0
    bpv = 2 * D + D // 2 + 2 * (D // G)
    n_eff = 4096 if a.op == "append" else N
    print(json.dumps({"op": a.op, "D": D, "dtype": a.dtype, "n": n_eff, "impl": a.impl, "ms_last": ms,
                      "ns_per_vec": ms * 1e6 / n_eff, "algorithmic_GBps": n_eff * bpv / (ms * 1e-3) / 1e9}))


if __name__ == "__main__":
    main()
