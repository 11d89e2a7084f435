#!/usr/bin/env python
"""Benchmark of the fused int4 KV-cache quantizer hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
    python bench.py --op decode --D 256 --dtype bf16 --n 524288 [--family gemm] [--sustain 4]     one kernel, one case

Workload: the Llama-3-70B-shaped cache (80 layers x 8 KV heads x D=128 fp16,
batch 4, prefix 32768).  One STEP is one pass of the whole hot path over one layer of that cache:

    kvq_encode   K and V of the layer: 2 x 1,048,576 vectors (bulk prefill encode, one launch, tensor-core kernel)
    kvq_append   one new vector per (K/V, head, batch) stream: 64 vectors written at the last row (matrix-vector kernel)
    kvq_decode   full-prefix read of the layer: 2,097,152 vectors back to fp16 (one launch, tensor-core kernel)

Successive steps rotate over distinct layer slots, so every buffer a kernel touches (0.15 - 0.54 GB)
is far larger than L2 and was last touched several launches ago.  The 80-layer sweep of the paper-shaped
model is 80 such steps.  With N > 1 ranks every rank runs its own layers (weak scaling, no collective:
vectors are independent and (layer, head) sharding needs no exchange).

Prints ONE JSON line.  `value` is algorithmic GB/s over the whole step (encode + append + decode
bytes / device time); the per-kernel figures, including encode ns/vec and prefix-decode GB/s as a
fraction of the measured HBM copy peak, are in `detail` and `roofline`.
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

D = 128
GROUP = 32
BYTES_PER_VEC = 2 * D + D // 2 + 2 * (D // GROUP)   # 328: fp16 row + packed row + fp16 scales
FALLBACK_HBM_GBS = 6650.0
METRIC = "hot-path algorithmic GB/s (encode + append + full-prefix decode; encode ns/vec and prefix-decode GB/s in detail)"
UNIT = "GB/s"


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def workload_shape():
    from paper_2605_05699_b200 import workloads as wl

    shp = wl.LLAMA3_70B
    streams = 2 * shp.kv_heads * shp.batch          # K and V streams of one layer: 64
    return shp, streams, shp.prefix                 # T = 32768 rows per stream


def slot_seed(rank: int, slot: int, n_slots: int) -> int:
    """Seed of layer slot `slot` on rank `rank`: ranks own disjoint layers (weak scaling, no exchange between them)."""
    return 5000 + 10 * (rank * n_slots + slot)


def max_over_ranks(ms: float, world: int, device) -> float:
    """The job's time is the slowest rank's: MAX all-reduce of a device-measured time (NCCL on GPUs, gloo in the CPU test)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist

    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        self.idx = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Median SM clock, maximum power and the throttle reasons seen over the samples taken between the two
        wall-clock times (the timed region); all samples if fewer than two fall inside."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        rows = []
        for line in out.splitlines():
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(f[1]), float(f[2]), float(f[3]),
                             [name for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9])
                              if v.lower().startswith("active")]))
            except ValueError:
                continue
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        inside = [r for r in rows if t_begin is not None and t_begin <= r[0] <= t_end]
        use = inside if len(inside) >= 2 else rows
        return {"sm_mhz": statistics.median(r[1] for r in use), "sm_max_mhz": max(r[2] for r in use),
                "reasons": sorted({n for r in use for n in r[4]}), "samples": len(use),
                "samples_inside_timed_region": len(inside), "power_w_max": max(r[3] for r in use)}


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------

def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2605_05699_b200 import binding as kb
    from paper_2605_05699_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    shp, S, T = workload_shape()
    N = S * T                                        # 2,097,152 vectors per step
    n_slots = 3
    plan = kb.Plan(D, GROUP, 70 + rank)
    lam = wl.make_lambda(2, D, 71 + rank, device=dev)             # one lambda row for K, one for V
    slots = []
    for s in range(n_slots):
        seed = slot_seed(rank, s, n_slots)
        xk = wl.make_vectors(N // 2, D, shp.dtype, "k_outlier", seed, device=dev)
        xv = wl.make_vectors(N // 2, D, shp.dtype, "gaussian", seed + 1, device=dev)
        x = torch.cat([xk, xv], 0)
        del xk, xv
        slots.append({
            "x": x,
            "x_new": wl.make_vectors(S, D, shp.dtype, "gaussian", seed + 2, device=dev),
            "packed": torch.empty(S, T, D // 2, dtype=torch.uint8, device=dev),
            "scales": torch.empty(S, T, D // GROUP, dtype=torch.float16, device=dev),
            "out": torch.empty(N, D, dtype=torch.float16, device=dev),
        })
    h = plan.handle
    rpl = N // 2                                     # rows per lambda row in the flat [N, D] view
    spl = S // 2                                     # streams per lambda row

    def step(sl, ev=None):
        if ev:
            ev[0].record()
        kb.kvq_encode(h, sl["x"], lam, sl["packed"], sl["scales"], rpl)
        if ev:
            ev[1].record()
        kb.kvq_append(h, sl["x_new"], lam, sl["packed"], sl["scales"], T - 1, spl)
        if ev:
            ev[2].record()
        kb.kvq_decode(h, sl["packed"], sl["scales"], lam, sl["out"], rpl)
        if ev:
            ev[3].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(slots[i % n_slots])
    barrier()

    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = kb.kvq_launch_count()
    barrier()
    wall0 = time.time()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(args.steps):
        step(slots[(args.warmup + i) % n_slots], evs[i])
    t1.record()
    barrier()
    wall1 = time.time()
    launches = kb.kvq_launch_count() - launches0
    clocks = sampler.stop(wall0, wall1) if rank == 0 else None
    ms_total = max_over_ranks(t0.elapsed_time(t1), world, dev)
    assert kb.kvq_plan_device_status(h) == 0, "a device-side wait timed out"

    n_first = min(100, args.steps)
    ms_first = evs[0][0].elapsed_time(evs[n_first - 1][3])        # the first steps: clocks still near boost
    enc_ms = [e[0].elapsed_time(e[1]) for e in evs]
    app_ms = [e[1].elapsed_time(e[2]) for e in evs]
    dec_ms = [e[2].elapsed_time(e[3]) for e in evs]

    # ---- end to end through the public API with HOST buffers (pinned), copies inside the timed region.  Every step
    # ---- copies its inputs in, runs the step and copies the result out; as in a serving loop the three stages of
    # ---- consecutive steps overlap (copy-in, compute and copy-out streams over two layer slots), so the rate is the
    # ---- slowest stage's, here a PCIe direction.
    e2e = None
    if rank == 0 or world > 1:
        e2e_steps = max(2, min(args.steps, 8))
        hx = torch.empty(N, D, dtype=torch.float16).pin_memory()
        hx.copy_(slots[0]["x"])
        hnew = torch.empty(S, D, dtype=torch.float16).pin_memory()
        hnew.copy_(slots[0]["x_new"])
        houts = [torch.empty(N, D, dtype=torch.float16).pin_memory() for _ in range(2)]
        s_in, s_run, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        ev = lambda: torch.cuda.Event(enable_timing=True)
        in_ready, run_done, out_done = [ev(), ev()], [ev(), ev()], [ev(), ev()]

        def e2e_run(n_steps):
            torch.cuda.synchronize()
            a, b = ev(), ev()
            a.record(s_in)
            for i in range(n_steps):
                k, sl = i % 2, slots[i % 2]
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(run_done[k])        # the step two back has read this slot's inputs
                    sl["x"].copy_(hx, non_blocking=True)
                    sl["x_new"].copy_(hnew, non_blocking=True)
                    in_ready[k].record(s_in)
                with torch.cuda.stream(s_run):
                    s_run.wait_event(in_ready[k])
                    if i >= 2:
                        s_run.wait_event(out_done[k])       # its result has left the device
                    step(sl)
                    run_done[k].record(s_run)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(run_done[k])
                    houts[k].copy_(sl["out"], non_blocking=True)
                    out_done[k].record(s_out)
            b.record(s_out)                                 # after the last result has reached the host buffer
            torch.cuda.synchronize()
            return a.elapsed_time(b)

        e2e_run(2)
        barrier()
        ms_e2e = max_over_ranks(e2e_run(e2e_steps), world, dev)
        barrier()
        step_bytes = (2 * N + S) * BYTES_PER_VEC
        e2e = {"value": world * e2e_steps * step_bytes / (ms_e2e * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": hx.numel() * 2 + hnew.numel() * 2, "d2h_bytes_per_step": houts[0].numel() * 2,
               "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps,
               "note": "copy-in, step and copy-out of consecutive steps overlap on three streams; bounded by one PCIe direction"}
        del hx, houts

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    copy_gbs = measure_sustained_copy(slots, dev)
    d256 = incr = sweep = c1 = c2 = c4 = sustained = None
    if not args.no_side:
        # the timed region of a short run (the default of the graded run is 20 steps, 6 ms) never reaches the board's power
        # cap: the same two kernels back to back for 0.6 s each show the capped regime
        if ms_total < 500.0:
            sustained = measure_sustained(kb, wl, dev, slots, plan, lam, rpl)
        d256 = measure_d256(kb, wl, dev)
        c1 = measure_config1(kb, wl, dev)
        c2 = measure_config2(kb, wl, dev)
        c4 = measure_config4(kb, wl, dev)
        incr = measure_incremental(kb, wl, dev, dec_avg_ms=sum(dec_ms) / len(dec_ms))
        sweep = measure_model_sweep(kb, wl, dev, shp.dtype, S, T)
    step_bytes = (2 * N + S) * BYTES_PER_VEC
    value = world * args.steps * step_bytes / (ms_total * 1e-3) / 1e9
    peak, peak_src = measured_peak()
    dec_avg = sum(dec_ms) / len(dec_ms)
    enc_avg = sum(enc_ms) / len(enc_ms)
    dec_gbs = N * BYTES_PER_VEC / (dec_avg * 1e-3) / 1e9
    enc_gbs = N * BYTES_PER_VEC / (enc_avg * 1e-3) / 1e9
    # The graded kernel is the full-prefix decode.  Its contraction is D^2 = 16384 flops per vector (one radix-2 step is taken
    # out of the 2 D^2 dense form; the encode runs two dense terms): ~0.012 ns/vec at the measured sustained tensor rate,
    # below the 0.051 ns/vec of bytes: HBM is the roof.
    roofline = {"bound": "hbm", "kernel": "kvq_decode_umma_kernel<128, fp16 out, 4-bit, radix-2> (full-prefix read, %d vectors per launch)" % N,
                "achieved": dec_gbs, "peak": peak, "unit": "GB/s", "frac": dec_gbs / peak,
                "peak_source": peak_src, "algorithmic_bytes_per_launch": N * BYTES_PER_VEC,
                "avg_launch_ms": dec_avg, "traffic": dram_traffic("decode"), "sustained": sustained,
                "sustained_copy_GBps": copy_gbs, "frac_of_sustained_copy": dec_gbs / copy_gbs,
                "sustained_copy_note": "a plain device copy of one layer buffer, back to back for 0.3 s in this run: the same "
                                       "power-capped regime as the timed region (peak above is the driver's burst copy)",
                "encode": {"kernel": "kvq_encode_umma_kernel<128, fp16 in> (%d vectors per launch)" % N, "achieved": enc_gbs,
                           "frac": enc_gbs / peak, "avg_launch_ms": enc_avg, "traffic": dram_traffic("encode")}}
    cpu = cpu_baseline_sample(target_seconds=12.0)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16 operands, f32 accumulate", "data": "synthetic",
        "config": {"workload": "llama-3-70b-shaped KV cache (config 5): one layer per step = encode 2x1,048,576 "
                               "vectors + append 64 + full-prefix decode 2,097,152 vectors, D=128 fp16 g=32",
                   "vectors_per_step": 2 * N + S, "bytes_per_vector": BYTES_PER_VEC, "io_dtype": "f16",
                   "l2": "every buffer (151-537 MB) exceeds L2; steps rotate over %d layer slots" % n_slots,
                   "parallelism": "layers sharded over ranks, no collective" if world > 1 else "single GPU"},
        "detail": {
            "encode_ns_per_vec": enc_avg * 1e6 / N, "encode_GBps": enc_gbs, "encode_frac_of_hbm_peak": enc_gbs / peak,
            "decode_ns_per_vec": dec_avg * 1e6 / N, "prefix_decode_GBps": dec_gbs,
            "prefix_decode_frac_of_hbm_peak": dec_gbs / peak, "prefix_decode_frac_of_8TBps": dec_gbs / 8000.0,
            "append_us": 1e3 * sum(app_ms) / len(app_ms),
            "value_first_%d_steps_GBps" % n_first: n_first * step_bytes / (ms_first * 1e-3) / 1e9,
            "power_note": "back to back for more than a few milliseconds the step runs at the board's 1000 W cap (sw_power_cap) "
                          "with the SM clock lowered to fit; roofline.sustained holds the two kernels in that regime",
            "encode_ms_min": min(enc_ms), "decode_ms_min": min(dec_ms),
            "model_sweep_decode_ms_80_layers": 80 * dec_avg,
            "model_sweep_measured": sweep,
            "paper_context": "paper: 24.6 ns/vec encode at D=128, ~50 ns/vec at D=256 on an Apple M1 GPU (fp32 in, Sec. 7.1)",
            "d256_bf16_gemma_shaped": d256,
            "config1": c1,
            "config2_qwen_shaped": c2,
            "config4": c4,
            "incremental_decode": incr,
        },
        "roofline": roofline,
        "cpu_baseline": cpu,
        "e2e": e2e,
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def measure_sustained_copy(slots, dev, seconds=0.3):
    """Outside the timed region: GB/s (read + write) of a plain device copy between two layer buffers, launched back to
    back for `seconds`: what the memory system delivers under the same power cap the timed steps run into."""
    import torch

    a, b = slots[0]["x"], slots[1]["out"]
    nbytes = 2 * a.numel() * a.element_size()
    for _ in range(3):
        b.copy_(a)
    torch.cuda.synchronize()
    reps = max(50, int(seconds / (nbytes / 6.0e12)))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        b.copy_(a)
    e1.record()
    torch.cuda.synchronize()
    return reps * nbytes / (e0.elapsed_time(e1) * 1e-3) / 1e9


def bytes_per_vector(Dh: int) -> int:
    return 2 * Dh + Dh // 2 + 2 * (Dh // GROUP)


def time_case(kb, wl, dev, Dh, dtype, Nv, kind, n_lambda=1, rpl=0, iters=12, warm=2, cold=False, seed=35):
    """Device time per kvq_encode and per kvq_decode launch of Nv vectors: `reps` launches queued back to back between two
    events on the launching stream, behind one more launch of the same call, so that neither the host's work for a launch
    (binding, tensor maps, the launch itself: 15-25 us that an event recorded on an idle stream would count as device time)
    nor an idle gap sits between the events; medians and minima over `iters` such measurements after `warm`.
    cold=False: the same buffers every launch (what fits stays in L2).  cold=True: the launches rotate over enough buffer
    sets to exceed 300 MB, more than twice the L2, so every launch reads from and writes to HBM."""
    import torch

    bpv = bytes_per_vector(Dh)
    n_sets = max(2, min(256, -(-300_000_000 // (Nv * bpv)))) if cold else 1
    reps = max(4, n_sets)
    plan = kb.Plan(Dh, GROUP, 33)
    lam = wl.make_lambda(n_lambda, Dh, seed - 1, device=dev)
    sets = []
    for k in range(n_sets):
        x = wl.make_vectors(Nv, Dh, dtype, kind, seed + k, device=dev)
        sets.append((x, plan.empty_packed(Nv, dev), plan.empty_scales(Nv, dev), torch.empty_like(x)))
    for x, pk, sc, out in sets:                      # the codes every decode reads
        kb.kvq_encode(plan.handle, x, lam, pk, sc, rpl)

    def encode(k):
        x, pk, sc, out = sets[k % n_sets]
        kb.kvq_encode(plan.handle, x, lam, pk, sc, rpl)

    def decode(k):
        x, pk, sc, out = sets[k % n_sets]
        kb.kvq_decode(plan.handle, pk, sc, lam, out, rpl)

    enc, dec = [], []
    for i in range(iters + warm):
        for fn, acc in ((encode, enc), (decode, dec)):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            fn(n_sets - 1)                           # in front: the stream is busy while the host queues the timed launches
            e0.record()
            for k in range(reps):
                fn(k)
            e1.record()
            torch.cuda.synchronize()
            if i >= warm:
                acc.append(e0.elapsed_time(e1) / reps)
    assert kb.kvq_plan_device_status(plan.handle) == 0
    plan.close()
    peak, _ = measured_peak()

    def stats(ms):
        med, mn = statistics.median(ms), min(ms)
        return {"us_median": 1e3 * med, "us_min": 1e3 * mn, "ns_per_vec": med * 1e6 / Nv, "GBps": Nv * bpv / (med * 1e-3) / 1e9,
                "frac_of_hbm_peak": Nv * bpv / (med * 1e-3) / 1e9 / peak}

    return {"encode": stats(enc), "decode": stats(dec), "launches_per_measurement": reps, "buffer_sets": n_sets}


def hot_and_cold(kb, wl, dev, Dh, dtype, Nv, kind, n_lambda=1, rpl=0, iters=20):
    bpv = bytes_per_vector(Dh)
    return {"vectors": Nv, "D": Dh, "io_dtype": dtype, "bytes_per_vector": bpv, "working_set_MB": Nv * bpv / 1e6,
            "hot_l2": time_case(kb, wl, dev, Dh, dtype, Nv, kind, n_lambda, rpl, iters, cold=False),
            "cold": time_case(kb, wl, dev, Dh, dtype, Nv, kind, n_lambda, rpl, iters, cold=True)}


def measure_config1(kb, wl, dev):
    """Config 1: one tensor of 4096 x 128 fp16 (1.3 MB in all): a launch-bound size, reported, not held to the roofline."""
    r = hot_and_cold(kb, wl, dev, 128, "f16", 4096, "c1")
    r["note"] = "4096 vectors: latency of one launch (the matrix-vector kernels serve calls of this size), not bandwidth"
    return r


def measure_config4(kb, wl, dev):
    """Config 4: the mixed-radix head dims, 65,536 vectors each, fp16, lognormal channel scales."""
    return {"D96": hot_and_cold(kb, wl, dev, 96, "f16", 65536, "lognormal"),
            "D160": hot_and_cold(kb, wl, dev, 160, "f16", 65536, "lognormal"),
            "note": "16-27 MB per launch: fits L2 when hot; cold = the launches rotate over more than 300 MB of buffer sets"}


def measure_config2(kb, wl, dev, steps=128):
    """Config 2, the Qwen2.5-1.5B-shaped decode loop: 28 layers x 2 KV heads x (K, V) = 112 streams of D=128 fp16, prefix 1024.
    Prefill encode of all streams in one call, then `steps` decode steps, each one kvq_append of 112 vectors (one launch, a
    lambda row per (layer, K/V)) and one full-prefix kvq_decode of the whole cache.  Device time per step between events."""
    import torch

    shp = wl.QWEN25_1P5B
    Dh, S, T0 = shp.head_dim, shp.streams, shp.prefix
    T_max = T0 + steps
    spl = shp.kv_heads
    plan = kb.Plan(Dh, GROUP, 77)
    lam = wl.make_lambda(S // spl, Dh, 21, device=dev)
    x = wl.make_vectors(S * T_max, Dh, shp.dtype, "k_outlier", 500, device=dev).view(S, T_max, Dh)
    packed = torch.zeros(S, T_max, Dh // 2, dtype=torch.uint8, device=dev)
    scales = torch.zeros(S, T_max, Dh // GROUP, dtype=torch.float16, device=dev)
    out = torch.empty(S * T_max, Dh, dtype=torch.float16, device=dev)
    xs = [x[:, T0 + t].contiguous() for t in range(steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    xp = x[:, :T0].contiguous()
    pp, sp = plan.empty_packed(S * T0, dev), plan.empty_scales(S * T0, dev)
    for rep in range(3):
        e0.record()
        kb.kvq_encode(plan.handle, xp.view(-1, Dh), lam, pp, sp, spl * T0)
        e1.record()
        torch.cuda.synchronize()
    prefill_ms = e0.elapsed_time(e1)
    packed[:, :T0] = pp.view(S, T0, -1)
    scales[:, :T0] = sp.view(S, T0, -1)
    ms = []
    for t in range(steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        kb.kvq_append(plan.handle, xs[t], lam, packed, scales, T0 + t, spl)
        kb.kvq_decode(plan.handle, packed.view(-1, Dh // 2), scales.view(-1, Dh // GROUP), lam, out, spl * T_max)
        b.record()
        ms.append((a, b))
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    plan.close()
    per = [a.elapsed_time(b) for a, b in ms][3:]
    peak, _ = measured_peak()
    bpv = bytes_per_vector(Dh)
    step_bytes = (S + S * T_max) * bpv
    med = statistics.median(per)
    return {"streams": S, "prefix": T0, "steps": steps, "vectors_decoded_per_step": S * T_max,
            "prefill_encode_us": 1e3 * prefill_ms, "prefill_encode_GBps": S * T0 * bpv / (prefill_ms * 1e-3) / 1e9,
            "step_us_median": 1e3 * med, "step_us_min": 1e3 * min(per), "step_bytes": step_bytes,
            "step_us_at_hbm_peak": step_bytes / (peak * 1e9) * 1e6, "step_GBps": step_bytes / (med * 1e-3) / 1e9,
            "note": "steps queued back to back on one stream; the 42 MB a step touches stay in L2 (hot), so the step is bound by two "
                    "launches, not by HBM; the whole [112, prefix + steps] cache is decoded every step, rows not yet written included"}


def measure_d256(kb, wl, dev):
    """Config 3, the Gemma-3-1B-shaped cache (26 layers x K,V, D=256 bf16): one encode and one decode launch over all layers
    (52 lambda rows) at prefix 256 / 1024 / 4096, and a launch of a million vectors that no cache can hold."""
    L = 2 * wl.GEMMA3_1B.layers
    res = {}
    for T in (256, 1024, 4096):
        res["prefix_%d" % T] = hot_and_cold(kb, wl, dev, 256, "bf16", L * T, "c1", L, T)
    big = L * 20480                                   # 1,064,960 vectors, 699 MB per launch
    res["hbm_bound_%d" % big] = {"vectors": big, "working_set_MB": big * bytes_per_vector(256) / 1e6,
                                 "cold": time_case(kb, wl, dev, 256, "bf16", big, "c1", L, 20480, iters=10, cold=True)}
    res["note"] = ("prefix sweep: 9-140 MB per launch, at or below the size of L2, and 9-70 us of device time of which 5-8 us are the "
                   "launch's fixed cost: not roofline numbers; the last entry is the D=256 roofline point")
    return res


def measure_sustained(kb, wl, dev, slots, plan, lam, rpl, seconds=0.6):
    """Outside the timed region: the step's two large kernels launched back to back for `seconds` each, with the SM clock
    sampled meanwhile: the power-capped regime that a short timed region never reaches."""
    import torch

    peak, _ = measured_peak()
    Nv = slots[0]["x"].shape[0]
    nbytes = Nv * BYTES_PER_VEC
    res = {}
    for name in ("decode", "encode"):
        def launch(i):
            sl = slots[i % len(slots)]
            if name == "decode":
                kb.kvq_decode(plan.handle, sl["packed"], sl["scales"], lam, sl["out"], rpl)
            else:
                kb.kvq_encode(plan.handle, sl["x"], lam, sl["packed"], sl["scales"], rpl)
        for i in range(3):
            launch(i)
        torch.cuda.synchronize()
        reps = max(100, int(seconds / 1.4e-4))
        sampler = ClockSampler(dev.index or 0)
        sampler.start()
        time.sleep(0.15)
        w0 = time.time()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(reps):
            launch(i)
        e1.record()
        torch.cuda.synchronize()
        w1 = time.time()
        clk = sampler.stop(w0, w1)
        us = 1e3 * e0.elapsed_time(e1) / reps
        res[name] = {"launches": reps, "us_per_launch": us, "GBps": nbytes / (us * 1e-6) / 1e9, "frac": nbytes / (us * 1e-6) / 1e9 / peak,
                     "sm_mhz_median": clk.get("sm_mhz"), "power_w_max": clk.get("power_w_max"), "reasons": clk.get("reasons"),
                     "us_times_mhz": None if clk.get("sm_mhz") is None else us * clk["sm_mhz"]}
    return res


def measure_model_sweep(kb, wl, dev, dtype, S, T, layers=80, sweeps=5):
    """Outside the timed region: the whole model's cache at once.  The int4 cache of all 80 layers (K and V of 64 streams x
    32,768 tokens each: 167,772,160 vectors, 12 GB) stays resident; one sweep = 80 full-prefix decodes, layer by layer, into
    one reused fp16 buffer, which is what one decode step of the model reads without a dequantized-prefix cache.  The
    prefill encode is timed per layer while the cache is being filled (its fp16 input is generated layer by layer)."""
    import torch

    N = S * T
    plan = kb.Plan(D, GROUP, 90)
    lam = wl.make_lambda(2 * layers, D, 91, device=dev)          # a lambda row per (layer, K / V)
    packed = torch.empty(layers, N, D // 2, dtype=torch.uint8, device=dev)
    scales = torch.empty(layers, N, D // GROUP, dtype=torch.float16, device=dev)
    enc_ms = []
    for l in range(layers):
        x = torch.cat([wl.make_vectors(N // 2, D, dtype, "k_outlier", 9000 + 2 * l, device=dev),
                       wl.make_vectors(N // 2, D, dtype, "gaussian", 9001 + 2 * l, device=dev)], 0)
        e = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        e[0].record()
        kb.kvq_encode(plan.handle, x, lam[2 * l:2 * l + 2], packed[l], scales[l], N // 2)
        e[1].record()
        torch.cuda.synchronize()
        enc_ms.append(e[0].elapsed_time(e[1]))
        del x
    out = torch.empty(N, D, dtype=torch.float16 if dtype == "f16" else torch.bfloat16, device=dev)
    ms = []
    for s in range(sweeps + 1):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        e[0].record()
        for l in range(layers):
            kb.kvq_decode(plan.handle, packed[l], scales[l], lam[2 * l:2 * l + 2], out, N // 2)
        e[1].record()
        torch.cuda.synchronize()
        if s > 0:
            ms.append(e[0].elapsed_time(e[1]))
    assert kb.kvq_plan_device_status(plan.handle) == 0
    plan.close()
    del packed, scales, out
    peak, _ = measured_peak()
    nbytes = layers * N * BYTES_PER_VEC
    med = statistics.median(ms)
    return {"layers": layers, "vectors": layers * N, "int4_cache_bytes": layers * N * (D // 2 + 2 * (D // GROUP)),
            "algorithmic_bytes_per_sweep": nbytes, "decode_sweep_ms": med, "decode_sweep_ms_all": ms,
            "decode_GBps": nbytes / (med * 1e-3) / 1e9, "decode_frac_of_hbm_peak": nbytes / (med * 1e-3) / 1e9 / peak,
            "ms_at_70pct_of_hbm_peak": nbytes / (0.7 * peak * 1e9) * 1e3,
            "prefill_encode_ms_sum_over_layers": sum(enc_ms), "prefill_encode_ms_per_layer_median": statistics.median(enc_ms),
            "note": "%d sweeps back to back after one warm-up sweep (each launch reads 151 MB it last saw 80 launches ago "
                    "and rewrites the 537 MB buffer); the encodes ran one by one with the input generation between them" % sweeps}


def measure_incremental(kb, wl, dev, dec_avg_ms, iters=20, window=16):
    """Outside the timed region: the window flush of Sec. 7.2 on the bench's cache shape (64 streams x 32,768 tokens,
    D=128 fp16): 16 new tokens per stream go into the int4 cache and the dequantized-prefix cache in one kvq_flush_block
    call, against re-decoding the whole prefix (the timed step's decode) once per generated token."""
    import torch

    shp, S, T = workload_shape()
    plan = kb.Plan(D, GROUP, 44)
    lam = wl.make_lambda(2, D, 45, device=dev)
    packed = torch.zeros(S, T, D // 2, dtype=torch.uint8, device=dev)
    scales = torch.zeros(S, T, D // GROUP, dtype=torch.float16, device=dev)
    dq = torch.zeros(S, T, D, dtype=torch.float16, device=dev)
    blocks = [wl.make_vectors(S * window, D, shp.dtype, "gaussian", 46 + i, device=dev).view(S, window, D) for i in range(4)]
    ms = []
    for i in range(iters + 3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pos0 = (i * 4099 * window) % (T - window)
        e0.record()
        kb.kvq_flush_block(plan.handle, blocks[i % 4], lam, packed, scales, dq, pos0, S // 2)
        e1.record()
        torch.cuda.synchronize()
        if i >= 3:
            ms.append(e0.elapsed_time(e1))
    # queued: the same calls without the synchronize between them (what a decode loop that keeps the stream busy sees)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        kb.kvq_flush_block(plan.handle, blocks[i % 4], lam, packed, scales, dq, (i * 4099 * window) % (T - window), S // 2)
    e1.record()
    torch.cuda.synchronize()
    queued_us = 1e3 * e0.elapsed_time(e1) / iters
    assert kb.kvq_plan_device_status(plan.handle) == 0
    plan.close()
    del packed, scales, dq
    flush_us = 1e3 * statistics.median(ms)
    return {"window_tokens": window, "streams": S, "flush_us": flush_us, "flush_us_queued": queued_us,
            "append_dispatch": measure_append_dispatch(kb, wl, dev, shp.dtype, S),
            "flush_us_per_generated_token": flush_us / window,
            "full_prefix_decode_us_per_generated_token": 1e3 * dec_avg_ms,
            "note": "one layer; the flush is one launch over %d vectors (launch-bound), independent of the prefix length" % (S * window)}


def measure_append_dispatch(kb, wl, dev, dtype, S, layers=80, T=1024, iters=20):
    """Outside the timed region: what the per-step append of a whole model (80 layers x 64 streams) costs by how it is
    dispatched -- one call per layer, the same 80 calls replayed as one CUDA graph (positions in device memory), and all
    5120 streams in ONE call (layers are streams of one cache, lambda row per layer and K / V)."""
    import torch

    plan = kb.Plan(D, GROUP, 47)
    lam = wl.make_lambda(2 * layers, D, 48, device=dev)
    x = wl.make_vectors(layers * S, D, dtype, "gaussian", 49, device=dev).view(layers, S, D)
    packed = torch.zeros(layers, S, T, D // 2, dtype=torch.uint8, device=dev)
    scales = torch.zeros(layers, S, T, D // GROUP, dtype=torch.float16, device=dev)
    pos = torch.zeros(1, dtype=torch.int64, device=dev)
    h = plan.handle

    def per_layer():
        for l in range(layers):
            kb.kvq_append_at(h, x[l], lam[2 * l:2 * l + 2], packed[l], scales[l], pos, S // 2)

    def one_call():
        kb.kvq_append_at(h, x.view(layers * S, D), lam, packed.view(layers * S, T, D // 2), scales.view(layers * S, T, D // GROUP),
                         pos, S // 2)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        per_layer()
        one_call()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        per_layer()
        pos.add_(1)

    def timed(fn):
        out = []
        for i in range(iters + 2):
            pos.fill_(i % T)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0 = time.perf_counter()
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            wall = 1e6 * (time.perf_counter() - t0)
            if i >= 2:
                out.append((1e3 * e0.elapsed_time(e1), wall))
        return statistics.median(o[0] for o in out), statistics.median(o[1] for o in out)

    eager = timed(per_layer)
    replay = timed(graph.replay)
    single = timed(one_call)
    assert kb.kvq_plan_device_status(h) == 0
    plan.close()
    return {"layers": layers, "streams_per_layer": S,
            "call_per_layer_us": eager[0], "call_per_layer_host_wall_us": eager[1],
            "cuda_graph_of_the_same_calls_us": replay[0], "cuda_graph_host_wall_us": replay[1],
            "one_call_all_layers_us": single[0], "one_call_host_wall_us": single[1],
            "note": "device time between events around the step / host wall time until the step has finished, medians; "
                    "kvq_append_at reads the row from device memory, so the graph is replayed as is for every position"}


def dram_traffic(which: str):
    """DRAM bytes of one full launch (dram__bytes_read.sum + dram__bytes_write.sum from a one-pass ncu capture of the bench's own
    launch size), as recorded by `python -m paper_2605_05699_b200.traffic`.  None when there is no record, or when the kernel's
    source file has changed since the counters were taken."""
    import hashlib

    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.json")) as f:
            rec = json.load(f)[which]
        with open(os.path.join(ROOT, "paper_2605_05699_b200", "csrc", rec["source"]), "rb") as f:
            if hashlib.sha256(f.read()).hexdigest()[:16] != rec["source_sha16"]:
                return None
        return int(rec["dram_bytes_read"]) + int(rec["dram_bytes_write"])
    except Exception:
        return None


# --------------------------------------------------------------------------------------------
# the oracle on the host cores: reported baseline and the reference arm
# --------------------------------------------------------------------------------------------

def _oracle_pass(n, seed):
    """One pass of the hot path in the oracle on n vectors (K-like half, V-like half): encode, append, decode."""
    import numpy as np

    from oracle import kvq_oracle as ko
    from paper_2605_05699_b200 import workloads as wl

    n -= n % 2
    half = n // 2
    x = np.concatenate([wl.raw_bits(wl.make_vectors(half, D, "f16", "k_outlier", seed)),
                        wl.raw_bits(wl.make_vectors(n - half, D, "f16", "gaussian", seed + 1))])
    lam = wl.make_lambda(2, D, seed + 2).numpy()
    sg = ko.signs(D, 70)
    xn = wl.raw_bits(wl.make_vectors(64, D, "f16", "gaussian", seed + 3))
    t0 = time.perf_counter()
    e = ko.encode(x, ko.F16, sg, lam, GROUP, rows_per_lambda=max(half, 1))
    pc = e["packed"][:64].reshape(64, 1, D // 2).copy()
    sc = e["scales"][:64].reshape(64, 1, D // GROUP).copy()
    ko.append(xn, ko.F16, sg, lam, GROUP, pc, sc, 0, 32)
    ko.decode(e["packed"], e["scales"], sg, lam, GROUP, ko.F16, rows_per_lambda=max(half, 1))
    dt = time.perf_counter() - t0
    return dt, (2 * n + 64) * BYTES_PER_VEC


def cpu_baseline_sample(target_seconds=12.0):
    from oracle import kvq_oracle as ko

    dt, nbytes = _oracle_pass(16384, 900)                      # calibration, also warms the library
    n = int(max(16384, min(4_000_000, 16384 * target_seconds / max(dt, 1e-3))))
    dt, nbytes = _oracle_pass(n, 901)
    return {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": ko.num_threads(), "kind": "oracle",
            "sample": "%d of the step's 2,097,152 vectors (half K-like, half V-like) + 64 appended: "
                      "oracle encode + append + decode, fp64 naive DFT, %.1f s" % (n, dt),
            "ns_per_vec_encode_plus_decode": dt * 1e9 / n}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import kvq_oracle as ko

    dt, _ = _oracle_pass(8192, 800)
    per_step = 60.0 / max(1, args.steps + args.warmup)          # keep the whole run near a minute
    n = int(max(8192, min(2_097_152, 8192 * per_step / max(dt, 1e-3))))
    for i in range(args.warmup):
        _oracle_pass(n, 810 + i)
    total_t, total_b = 0.0, 0
    for i in range(args.steps):
        t, b = _oracle_pass(n, 820 + i)
        total_t += t
        total_b += b
    value = total_b / total_t / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(args.gpus),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "llama-3-70b-shaped KV cache (config 5): bounded sample of %d vectors of the "
                               "step's 2,097,152 per step, D=128 fp16 g=32" % n},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": ko.num_threads(), "kind": "oracle",
                         "sample": "%d vectors per step, encode + append + decode" % n},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------
# one kernel, one case: the command that goes under a profiler, and the back-to-back (power-capped) probe
# --------------------------------------------------------------------------------------------

FAMILY = {"auto": 0, "fft": 1, "gemm": 2, "matvec": 3}


def run_case(args):
    """`--op encode|decode|append|flush|copy`: runs ONE kernel on one fixed case a few times and prints one JSON line with the
    CUDA-event time of the last launch (never quote a time taken under a profiler).  With `--sustain SECONDS` the op is
    launched back to back for that long over three buffer sets, timed in chunks of 200 launches, while nvidia-smi is sampled:
    the board's power cap bounds the large kernels in steady state (`--op copy` is a plain device copy, the reference)."""
    import torch

    from paper_2605_05699_b200 import binding as kb
    from paper_2605_05699_b200 import workloads as wl

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    Dh, Nv, fam = args.D, args.n, FAMILY[args.family]
    n_lambda = max(1, args.n_lambda)
    rpl = (Nv + n_lambda - 1) // n_lambda if n_lambda > 1 else 0
    bpv = bytes_per_vector(Dh)
    plan = kb.Plan(Dh, GROUP, 3)
    lam = wl.make_lambda(n_lambda, Dh, 12, device=dev)
    n_sets = 3 if args.sustain > 0 else 1
    sets = []
    for i in range(n_sets):
        x = wl.make_vectors(Nv, Dh, args.dtype, args.kind, 11 + i, device=dev)
        sets.append((x, plan.empty_packed(Nv, dev), plan.empty_scales(Nv, dev), torch.empty_like(x)))
    # the compressed input of decode comes from the fp32 register-FFT encoder
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_FFT, fam)
    for x, pk, sc, out in sets:
        kb.kvq_encode(plan.handle, x, lam, pk, sc, rpl)
    kb.kvq_plan_set_impl(plan.handle, fam, fam)
    torch.cuda.synchronize()

    def launch(i):
        x, pk, sc, out = sets[i % n_sets]
        if args.op == "encode":
            kb.kvq_encode(plan.handle, x, lam, pk, sc, rpl)
        elif args.op == "decode":
            kb.kvq_decode(plan.handle, pk, sc, lam, out, rpl)
        elif args.op == "append":
            kb.kvq_append(plan.handle, x[:4096], lam[:1], pk.view(4096, -1, Dh // 2), sc.view(4096, -1, Dh // GROUP), 1)
        elif args.op == "flush":   # the window flush: 64 streams x 16 new tokens into caches of n / 64 rows per stream, one launch
            kb.kvq_flush_block(plan.handle, x[:1024].view(64, 16, Dh), lam[:1], pk.view(64, -1, Dh // 2), sc.view(64, -1, Dh // GROUP),
                               out.view(64, -1, Dh), 16)
        else:
            out.copy_(sets[(i + 1) % n_sets][0])

    base = {"op": args.op, "D": Dh, "io_dtype": args.dtype, "family": args.family, "n_lambda": n_lambda}
    if args.sustain > 0:
        if args.op in ("append", "flush"):
            raise SystemExit("--sustain takes encode, decode or copy")
        time.sleep(1.0)
        sampler = ClockSampler(0)
        sampler.start()
        chunks = []
        w0 = time.time()
        while time.time() < w0 + args.sustain:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(200):
                launch(i)
            e1.record()
            torch.cuda.synchronize()
            chunks.append(1e3 * e0.elapsed_time(e1) / 200)
        w1 = time.time()
        clk = sampler.stop(w0 + 0.5 * (w1 - w0), w1)
        assert kb.kvq_plan_device_status(plan.handle) == 0
        nbytes = Nv * bpv if args.op != "copy" else 2 * Nv * 2 * Dh
        tail = sorted(chunks[len(chunks) // 2:])
        steady = tail[len(tail) // 2]
        base.update({"n": Nv, "seconds": args.sustain, "us_per_launch_first_chunk": chunks[0], "us_per_launch_steady": steady,
                     "GBps_steady": nbytes / (steady * 1e-6) / 1e9, "bytes_per_launch": nbytes, "clocks_second_half": clk})
        print(json.dumps(base))
        return
    if args.op == "copy":
        raise SystemExit("--op copy is for --sustain")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(max(1, args.reps)):
        e0.record()
        launch(0)
        e1.record()
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    assert kb.kvq_plan_device_status(plan.handle) == 0
    n_eff = 4096 if args.op == "append" else 1024 if args.op == "flush" else Nv
    base.update({"n": n_eff, "ms_last": ms, "ns_per_vec": ms * 1e6 / n_eff, "algorithmic_GBps": n_eff * bpv / (ms * 1e-3) / 1e9})
    print(json.dumps(base))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)   # 0.6 s of back-to-back steps: long enough to sample the clocks under load
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-side", action="store_true",
                    help="leave out the measurements beside the timed region (D=256, window flush, 80-layer sweep): for a launch list")
    # one kernel on one case (see run_case): a profiler's command line
    ap.add_argument("--op", choices=["encode", "decode", "append", "flush", "copy"], default=None)
    ap.add_argument("--D", type=int, default=128)
    ap.add_argument("--dtype", choices=["f16", "bf16"], default="f16")
    ap.add_argument("--n", type=int, default=1 << 20)
    ap.add_argument("--n-lambda", type=int, default=1)
    ap.add_argument("--family", choices=["auto", "fft", "gemm", "matvec"], default="auto")
    ap.add_argument("--kind", default="k_outlier")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--sustain", type=float, default=0.0, help="with --op: seconds of back-to-back launches with nvidia-smi sampling")
    args = ap.parse_args()
    if args.op is not None:
        return run_case(args)
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
