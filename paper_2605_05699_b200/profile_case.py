"""Runs one small, fixed case of one libkvq kernel a few times: the command to put under ncu.

    python -m paper_2605_05699_b200.profile_case --op decode --D 128 --dtype f16 --n 1048576 --impl auto --reps 3

The case is sized for a profiler capture: inputs and outputs larger than L2, well under a GB on the
device, a handful of launches, nothing else running.  It prints the CUDA-event time of the last launch
so the same command doubles as a quick timing probe (never quote a time taken under a profiler).

    python -m paper_2605_05699_b200.profile_case --op encode --n 2097152 --sustain 4

With ``--sustain SECONDS`` the op is launched back to back for that long over three buffer sets (no profiler), timed
in chunks of 200 launches, while ``nvidia-smi`` is sampled every 100 ms: the board's power cap, not HBM, bounds the
kernels in steady state, and this is the command that shows it (``--op copy`` is a plain device copy of the same
input, the reference).
"""
from __future__ import annotations

import argparse
import json
import subprocess
import tempfile
import time

import torch

from . import binding as kb
from . import workloads as wl

IMPL = {"auto": kb.KVQ_IMPL_AUTO, "fft": kb.KVQ_IMPL_FFT, "gemm": kb.KVQ_IMPL_GEMM, "matvec": kb.KVQ_IMPL_MATVEC}

SMI_QUERY = "clocks.sm,power.draw,clocks_event_reasons.sw_power_cap,clocks_event_reasons.hw_slowdown,clocks_event_reasons.sw_thermal_slowdown"


def sustain(a):
    """Back-to-back launches for a.sustain seconds; prints one JSON line with chunk times and the sampled clocks."""
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    D, G, N = a.D, wl.GROUP, a.n
    plan = kb.Plan(D, G, 3)
    lam = wl.make_lambda(2, D, 12, device=dev)
    sets = []
    for s in range(3):
        x = wl.make_vectors(N, D, a.dtype, a.kind, 11 + s, device=dev)
        sets.append((x, plan.empty_packed(N), plan.empty_scales(N), torch.empty_like(x)))
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_FFT, kb.KVQ_IMPL_FFT)
    for x, p, s, o in sets:
        kb.kvq_encode(plan.handle, x, lam, p, s, N // 2)
    kb.kvq_plan_set_impl(plan.handle, IMPL[a.impl], IMPL[a.impl])
    torch.cuda.synchronize()
    time.sleep(1.0)

    def launch(i):
        x, p, s, o = sets[i % 3]
        if a.op == "encode":
            kb.kvq_encode(plan.handle, x, lam, p, s, N // 2)
        elif a.op == "decode":
            kb.kvq_decode(plan.handle, p, s, lam, o, N // 2)
        else:
            o.copy_(sets[(i + 1) % 3][0])

    with tempfile.TemporaryFile("w+") as log:
        smi = subprocess.Popen(["nvidia-smi", "-i", "0", "--query-gpu=" + SMI_QUERY, "--format=csv,noheader,nounits", "-lms", "100"], stdout=log)
        chunks = []
        t_end = time.time() + a.sustain
        while time.time() < t_end:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(200):
                launch(i)
            e1.record()
            torch.cuda.synchronize()
            chunks.append(1e3 * e0.elapsed_time(e1) / 200)
        smi.terminate()
        smi.wait()
        log.seek(0)
        rows = [r.split(", ") for r in log.read().splitlines() if r.strip()]
    assert kb.kvq_plan_device_status(plan.handle) == 0
    tail = rows[len(rows) // 2:]
    bpv = 2 * D + D // 2 + 2 * (D // G)
    nbytes = N * bpv if a.op != "copy" else 2 * N * 2 * D
    steady = sorted(chunks[len(chunks) // 2:])[len(chunks[len(chunks) // 2:]) // 2]
    print(json.dumps({"op": a.op, "D": D, "dtype": a.dtype, "n": N, "impl": a.impl, "seconds": a.sustain,
                      "us_per_launch_first_chunk": chunks[0], "us_per_launch_steady": steady,
                      "GBps_steady": nbytes / (steady * 1e-6) / 1e9, "bytes_per_launch": nbytes,
                      "sm_mhz_steady": sorted(float(r[0]) for r in tail)[len(tail) // 2],
                      "power_w_steady": sorted(float(r[1]) for r in tail)[len(tail) // 2],
                      "sw_power_cap": sorted(set(r[2] for r in tail)), "hw_slowdown": sorted(set(r[3] for r in tail)),
                      "sw_thermal_slowdown": sorted(set(r[4] for r in tail))}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", choices=["encode", "decode", "append", "flush", "copy"], default="decode")
    ap.add_argument("--D", type=int, default=128)
    ap.add_argument("--dtype", choices=["f16", "bf16"], default="f16")
    ap.add_argument("--n", type=int, default=1 << 20)
    ap.add_argument("--impl", choices=list(IMPL), default="auto")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--kind", default="k_outlier")
    ap.add_argument("--sustain", type=float, default=0.0, help="seconds of back-to-back launches with nvidia-smi sampling")
    a = ap.parse_args()
    if a.sustain > 0:
        if a.op in ("append", "flush"):
            ap.error("--sustain takes encode, decode or copy")
        return sustain(a)
    if a.op == "copy":
        ap.error("--op copy is for --sustain")

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
        elif a.op == "append":
            kb.kvq_append(plan.handle, x[:4096], lam, packed.view(4096, -1, D // 2), scales.view(4096, -1, D // G), 1)
        else:   # the window flush: 64 streams x 16 new tokens into caches of n / 64 rows per stream, one launch
            kb.kvq_flush_block(plan.handle, x[:1024].view(64, 16, D), lam, packed.view(64, -1, D // 2), scales.view(64, -1, D // G),
                               out.view(64, -1, D), 16)
        e1.record()
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    assert kb.kvq_plan_device_status(plan.handle) == 0
    bpv = 2 * D + D // 2 + 2 * (D // G)
    n_eff = 4096 if a.op == "append" else 1024 if a.op == "flush" else N
    print(json.dumps({"op": a.op, "D": D, "dtype": a.dtype, "n": n_eff, "impl": a.impl, "ms_last": ms,
                      "ns_per_vec": ms * 1e6 / n_eff, "algorithmic_GBps": n_eff * bpv / (ms * 1e-3) / 1e9}))


if __name__ == "__main__":
    main()
