"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded inputs."""
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


def bits(t):
    return wl.raw_bits(t)


def gpu_encode(plan, x, lam, rows_per_lambda=0):
    N = x.shape[0]
    packed, scales = plan.empty_packed(N), plan.empty_scales(N)
    kb.kvq_encode(plan.handle, x, lam, packed, scales, rows_per_lambda)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    return packed, scales


def gpu_decode(plan, packed, scales, lam, dtype, rows_per_lambda=0):
    N = packed.shape[0]
    out = torch.empty(N, plan.D, dtype=wl.torch_dtype(dtype), device="cuda")
    kb.kvq_decode(plan.handle, packed, scales, lam, out, rows_per_lambda)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    return out


def gpu_decode_raw(plan, packed, scales, lam, dtype, rows_per_lambda=0):
    """gpu_decode without the finiteness assumption of the callers that follow it with check_decode on every row."""
    out = torch.empty(packed.shape[0], plan.D, dtype=wl.torch_dtype(dtype), device="cuda")
    kb.kvq_decode(plan.handle, packed, scales, lam, out, rows_per_lambda)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0         # no bounded wait ran out, nothing else to report
    return out


IMPL = {"auto": kb.KVQ_IMPL_AUTO, "fft": kb.KVQ_IMPL_FFT, "gemm": kb.KVQ_IMPL_GEMM, "matvec": kb.KVQ_IMPL_MATVEC}


def run_case(D, dtype, N, kind, seed, n_lambda=1, rows_per_lambda=0, plan_seed=None, enc_impl="auto", dec_impl="auto"):
    """Encode on GPU vs oracle; decode the ORACLE's compressed data on GPU vs oracle; GPU round trip."""
    plan = kb.Plan(D, G, seed if plan_seed is None else plan_seed)
    kb.kvq_plan_set_impl(plan.handle, IMPL[enc_impl], IMPL[dec_impl])
    sg = plan.signs()
    assert np.array_equal(sg, ko.signs(D, plan.seed))  # two independent implementations of the sign stream
    x = wl.make_vectors(N, D, dtype, kind, seed)
    lam = wl.make_lambda(n_lambda, D, seed + 1)
    ora = ko.encode(bits(x), DT[dtype], sg, lam.numpy(), G, rows_per_lambda, want_v=True)
    xd, lamd = x.cuda(), lam.cuda()
    packed, scales = gpu_encode(plan, xd, lamd, rows_per_lambda)
    label = "D=%d %s N=%d" % (D, dtype, N)
    enc = parity.check_encode(packed.cpu().numpy(), bits(scales), ora, G, label + " encode")
    # decode parity on the oracle's own compressed representation
    ob, o64 = ko.decode(ora["packed"], ora["scales"], sg, lam.numpy(), G, DT[dtype], rows_per_lambda, want_f64=True)
    pk_o = torch.from_numpy(ora["packed"]).cuda()
    sc_o = torch.from_numpy(ora["scales"].view(np.int16)).view(torch.float16).cuda()
    out = gpu_decode(plan, pk_o, sc_o, lamd, dtype, rows_per_lambda)
    dec = parity.check_decode(bits(out), ob, o64, DT[dtype], label + " decode")
    # GPU round trip stays close to the input (4-bit noise level, sanity only)
    rt = gpu_decode(plan, packed, scales, lamd, dtype, rows_per_lambda).float().cpu().numpy()
    xin = x.float().numpy()
    rel = parity.rel_l2_rows(rt, xin)
    assert np.median(rel) < 0.2
    plan.close()
    return enc, dec


# ---- config 1: one tensor, 4096 x 128 fp16, outlier channels, lambda U(0.5, 2) -------------

def test_config1_single_tensor_d128_f16():
    enc, dec = run_case(128, "f16", 4096, "c1", 1001)
    assert enc["mismatches"] <= 52  # 99.99 % of 524288 codes


# ---- both decode kernel families at D = 128 fp16: the fp32 register FFT and the tcgen05 DFT-as-GEMM

@pytest.mark.parametrize("dec_impl", ["fft", "gemm"])
@pytest.mark.parametrize("N,n_lambda,rpl,kind", [(4096, 1, 0, "c1"), (1000, 4, 333, "k_outlier"), (1, 1, 0, "gaussian"),
                                                 (129, 1, 0, "gaussian"), (70000, 7, 10000, "k_outlier")])
def test_decode_kernel_families_d128_f16(dec_impl, N, n_lambda, rpl, kind):
    enc, dec = run_case(128, "f16", N, kind, 8000 + N, n_lambda=n_lambda, rows_per_lambda=rpl, dec_impl=dec_impl)
    if dec_impl == "fft":
        assert dec["rel_l2_plain_max"] < 1e-3  # fp32 arithmetic: far inside the tolerance even without the tie rule


# ---- both encode kernel families at D = 128: the fp32 register FFT and the tcgen05 DFT-as-GEMM with split W

@pytest.mark.parametrize("enc_impl", ["fft", "gemm"])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("N,n_lambda,rpl,kind", [(4096, 1, 0, "c1"), (1000, 4, 333, "k_outlier"), (1, 1, 0, "gaussian"),
                                                 (129, 1, 0, "gaussian"), (70000, 7, 10000, "k_outlier")])
def test_encode_kernel_families_d128(enc_impl, dtype, N, n_lambda, rpl, kind):
    enc, dec = run_case(128, dtype, N, kind, 9000 + N, n_lambda=n_lambda, rows_per_lambda=rpl, enc_impl=enc_impl, dec_impl="fft")
    assert enc["mismatches"] <= max(2, int(1e-4 * N * 128))


@pytest.mark.parametrize("rpl", [128, 200, 640])
def test_many_lambda_rows_rebuild_the_gemm_operands_in_flight(rpl):
    # every few tiles a new lambda row: the tensor-core kernels rebuild their B operand while other tiles are in flight
    N = 60000
    n_lambda = (N + rpl - 1) // rpl
    for rep in range(2):
        enc, dec = run_case(128, "f16", N, "k_outlier", 9500 + rpl + rep, n_lambda=n_lambda, rows_per_lambda=rpl,
                            enc_impl="gemm", dec_impl="gemm")


@pytest.mark.parametrize("D,rpl", [(128, 128), (128, 200), (64, 640), (96, 384), (160, 128), (160, 333)])
def test_bf16_output_on_the_tensor_cores_with_many_lambda_rows(D, rpl):
    # two-term operands (a_hi + a_lo, W_hi + W_lo), two A stages (one at D = 160), B rebuilt every few tiles
    N = 40000
    run_case(D, "bf16", N, "k_outlier", 9700 + D + rpl, n_lambda=(N + rpl - 1) // rpl, rows_per_lambda=rpl,
             enc_impl="gemm", dec_impl="gemm")


def test_lambda_scale_does_not_matter_to_the_gemm_encode():
    # lambda rows far from 1: the power-of-two lift keeps the split terms of W inside fp16's normal range
    for shift in (-12, 9):
        D, N = 128, 2048
        plan = kb.Plan(D, G, 31)
        kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_GEMM, kb.KVQ_IMPL_FFT)
        sg = plan.signs()
        x = wl.make_vectors(N, D, "f16", "k_outlier", 77)
        lam = wl.make_lambda(1, D, 78) * (2.0 ** shift)
        ora = ko.encode(bits(x), ko.F16, sg, lam.numpy(), G, want_v=True)
        packed, scales = gpu_encode(plan, x.cuda(), lam.cuda())
        parity.check_encode(packed.cpu().numpy(), bits(scales), ora, G, "gemm encode, lambda x 2^%d" % shift)
        plan.close()


def test_gemm_encode_serves_large_appends():
    # append of many streams goes through the same tensor-core kernel with scattered output rows
    D, S, T = 128, 5000, 3
    plan = kb.Plan(D, G, 6)
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_GEMM, kb.KVQ_IMPL_AUTO)
    x = wl.make_vectors(S, D, "f16", "k_outlier", 19)
    lam = wl.make_lambda(5, D, 20)
    packed = torch.full((S, T, D // 2), 0xAB, dtype=torch.uint8, device="cuda")
    scales = torch.full((S, T, D // G), 1.25, dtype=torch.float16, device="cuda")
    kb.kvq_append(plan.handle, x.cuda(), lam.cuda(), packed, scales, 1, 1000)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    assert bool((packed[:, [0, 2]] == 0xAB).all()) and bool((scales[:, [0, 2]] == 1.25).all())
    ora = ko.encode(bits(x), ko.F16, plan.signs(), lam.numpy(), G, 1000, want_v=True)
    parity.check_encode(packed[:, 1].contiguous().cpu().numpy(), bits(scales[:, 1].contiguous()), ora, G, "gemm append")
    plan.close()


def test_gemm_kernels_are_refused_where_they_are_not_built():
    for D, dtype, nbits in [(160, torch.bfloat16, 8)]:
        plan = kb.Plan(D, G, 1, nbits)
        kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_AUTO, kb.KVQ_IMPL_GEMM)
        pk, sc = plan.empty_packed(8), plan.empty_scales(8)
        out = torch.empty(8, D, dtype=dtype, device="cuda")
        with pytest.raises(kb.KvqError) as e:
            kb.kvq_decode(plan.handle, pk, sc, torch.ones(D, device="cuda"), out)
        assert e.value.status == kb.KVQ_ERR_UNSUPPORTED_DIM
        plan.close()
    for D, dtype, nbits in [(160, torch.bfloat16, 8), (256, torch.bfloat16, 8)]:     # byte codes from bf16: a three-term B does not fit
        plan = kb.Plan(D, G, 1, nbits)
        kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_GEMM, kb.KVQ_IMPL_AUTO)
        x = torch.zeros(8, D, dtype=dtype, device="cuda")
        with pytest.raises(kb.KvqError) as e:
            kb.kvq_encode(plan.handle, x, torch.ones(D, device="cuda"), plan.empty_packed(8), plan.empty_scales(8))
        assert e.value.status == kb.KVQ_ERR_UNSUPPORTED_DIM
        plan.close()


def test_lambda_scale_does_not_matter_to_the_gemm_decode():
    # lambda rows far from 1 (all channels x 2^-12 or x 2^9): the power-of-two normalisation keeps fp16 operands in range
    for shift in (-12, 9):
        D, N = 128, 2048
        plan = kb.Plan(D, G, 31)
        kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_FFT, kb.KVQ_IMPL_GEMM)
        sg = plan.signs()
        x = wl.make_vectors(N, D, "f16", "k_outlier", 77)
        lam = wl.make_lambda(1, D, 78) * (2.0 ** shift)
        ora = ko.encode(bits(x), ko.F16, sg, lam.numpy(), G, want_v=True)
        ob, o64 = ko.decode(ora["packed"], ora["scales"], sg, lam.numpy(), G, ko.F16, want_f64=True)
        pk = torch.from_numpy(ora["packed"]).cuda()
        sc = torch.from_numpy(ora["scales"].view(np.int16)).view(torch.float16).cuda()
        out = gpu_decode(plan, pk, sc, lam.cuda(), "f16")
        parity.check_decode(bits(out), ob, o64, ko.F16, "gemm decode, lambda x 2^%d" % shift)
        plan.close()


# ---- D = 256 decode on the tensor cores: CTA pairs, one term for fp16 output, split operands for bf16 output

@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("N,n_lambda,rpl,kind", [(4096, 1, 0, "c1"), (1000, 4, 333, "k_outlier"), (1, 1, 0, "gaussian"),
                                                 (129, 1, 0, "gaussian"), (40000, 9, 4500, "k_outlier"), (30000, 150, 200, "c1"),
                                                 (30000, 235, 128, "c1"), (40000, 105, 384, "k_outlier")])
def test_gemm_kernels_d256(dtype, N, n_lambda, rpl, kind):
    enc, dec = run_case(256, dtype, N, kind, 9700 + N, n_lambda=n_lambda, rows_per_lambda=rpl, enc_impl="gemm", dec_impl="gemm")
    assert enc["mismatches"] <= max(2, int(1e-4 * N * 256))
    if dtype == "bf16":
        assert dec["rows_needing_tie_rule"] < 0.02


# ---- static lambda calibration (Sec. 7.1): lambda_c = 1 / max over the calibration vectors of |SRFT(x)_c|

@pytest.mark.parametrize("D,dtype", [(64, "f16"), (96, "f16"), (128, "f16"), (128, "bf16"), (160, "f16"), (256, "f16"), (256, "bf16")])
@pytest.mark.parametrize("N", [1, 700, 40000])
def test_calibrate_lambda_matches_the_oracle(D, dtype, N):
    plan = kb.Plan(D, G, 50 + D)
    sg = plan.signs()
    x = wl.make_vectors(N, D, dtype, "k_outlier", 60 + D + N)
    lam_o, amax_o = ko.calibrate_lambda(bits(x), DT[dtype], sg)
    lam = torch.full((D,), -1.0, dtype=torch.float32, device="cuda")
    kb.kvq_calibrate_lambda(plan.handle, x.cuda(), lam)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    got = lam.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got)) and np.all(got > 0)
    # fp32 accumulation of exact products against fp64.  The error of a coefficient is relative to the vector's norm (the
    # transform is orthonormal), not to the coefficient, which may be a small remainder of cancelling terms.
    xnorm = float(np.linalg.norm(x.double().numpy(), axis=1).max())
    assert np.abs(1.0 / got - amax_o).max() <= 2e-6 * xnorm
    if N >= 700:   # with many vectors every channel's maximum is of the order of the norms, and lambda itself agrees
        assert np.abs(got / lam_o - 1.0).max() <= 1e-4
    # used as lambda, every rescaled channel stays within [-1, 1]: no group scale exceeds fp16(1 / 7) by more than rounding
    packed, scales = gpu_encode(plan, x.cuda(), lam)
    assert float(scales.float().max()) <= (1.0 / 7.0) * (1.0 + 2e-3)
    plan.close()


@pytest.mark.parametrize("D,dtype", [(128, "f16"), (256, "bf16"), (160, "f16")])
def test_gemm_decode_with_the_calibrated_lambda(D, dtype):
    """Static lambda as the library itself calibrates it on K-like data with outlier channels (Sec. 5.1 item 1,
    Sec. 7.1), then used by the tensor-core encode and decode: codes, scales and reconstruction against the oracle run with
    the same lambda."""
    odt = DT[dtype]
    N = 5000
    plan = kb.Plan(D, G, 70 + D)
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_GEMM, kb.KVQ_IMPL_GEMM)
    sg = plan.signs()
    x = wl.make_vectors(N, D, dtype, "k_outlier", 71 + D)
    lam = torch.empty(D, dtype=torch.float32, device="cuda")
    kb.kvq_calibrate_lambda(plan.handle, x.cuda(), lam)
    torch.cuda.synchronize()
    lam_h = lam.cpu().numpy().astype(np.float64).reshape(1, D)
    print("calibrated lambda spans a factor of %.1f" % (lam_h.max() / lam_h.min()))
    packed, scales = gpu_encode(plan, x.cuda(), lam.view(1, D))
    ora = ko.encode(bits(x), odt, sg, lam_h, G, want_v=True)
    parity.check_encode(packed.cpu().numpy(), bits(scales), ora, G, "encode with the calibrated lambda", min_agree=0.9995)
    ob, o64 = ko.decode(ora["packed"], ora["scales"], sg, lam_h, G, odt, want_f64=True)
    out = gpu_decode_raw(plan, torch.from_numpy(ora["packed"]).cuda(),
                         torch.from_numpy(ora["scales"].view(np.int16)).view(torch.float16).cuda(), lam.view(1, D), dtype)
    parity.check_decode(bits(out), ob, o64, odt, "decode with the calibrated lambda")
    plan.close()


def test_calibrate_lambda_edge_cases():
    plan = kb.Plan(128, G, 3)
    lam = torch.full((128,), -1.0, dtype=torch.float32, device="cuda")
    kb.kvq_calibrate_lambda(plan.handle, torch.empty(0, 128, dtype=torch.float16, device="cuda"), lam)
    torch.cuda.synchronize()
    assert bool((lam == 1.0).all())                       # no vectors: lambda = 1
    kb.kvq_calibrate_lambda(plan.handle, torch.zeros(300, 128, dtype=torch.float16, device="cuda"), lam)
    torch.cuda.synchronize()
    assert bool((lam == 1.0).all())                       # channels that carry nothing: lambda = 1
    plan.close()
    p160 = kb.Plan(160, G, 3)
    with pytest.raises(kb.KvqError) as e:
        kb.kvq_calibrate_lambda(p160.handle, torch.zeros(8, 160, dtype=torch.bfloat16, device="cuda"), torch.empty(160, device="cuda"))
    assert e.value.status == kb.KVQ_ERR_UNSUPPORTED_DIM
    p160.close()


# ---- every head dim and dtype, ragged N (several tiles plus a tail), lambda rows that straddle tiles

@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("D", [64, 96, 128, 160, 256])
def test_all_dims_ragged_with_straddling_lambda_rows(D, dtype):
    run_case(D, dtype, 1000, "k_outlier", 2000 + D, n_lambda=4, rows_per_lambda=333, enc_impl="fft", dec_impl="fft")


# the tensor-core kernels of D <= 160, both dtypes, both directions
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("D", [64, 96, 128, 160])
@pytest.mark.parametrize("N,n_lambda,rpl", [(1000, 4, 333), (20000, 1, 0), (129, 1, 0)])
def test_gemm_kernels_all_dims(D, dtype, N, n_lambda, rpl):
    run_case(D, dtype, N, "k_outlier", 2100 + D + N, n_lambda=n_lambda, rows_per_lambda=rpl, enc_impl="gemm", dec_impl="gemm")


@pytest.mark.parametrize("N", [1, 31, 32, 33, 4100])
def test_small_and_ragged_sizes(N):
    run_case(128, "f16", N, "gaussian", 3000 + N)


def test_empty_input_is_a_noop():
    plan = kb.Plan(128, G, 1)
    x = torch.empty(0, 128, dtype=torch.float16, device="cuda")
    lam = torch.ones(128, device="cuda")
    pk, sc = plan.empty_packed(0), plan.empty_scales(0)
    kb.kvq_encode(plan.handle, x, lam, pk, sc)
    kb.kvq_decode(plan.handle, pk, sc, lam, x)
    torch.cuda.synchronize()


# ---- config 4: mixed-radix head dims, 65536 vectors each ------------------------------------

@pytest.mark.parametrize("impl", ["fft", "gemm"])
@pytest.mark.parametrize("D", [96, 160])
def test_config4_mixed_radix(D, impl):
    # the register FFT takes the radix-3 / radix-5 path; the tensor-core kernels contract with the D x D matrix directly
    run_case(D, "f16", 65536, "lognormal", 4000 + D, enc_impl=impl, dec_impl=impl)


# ---- config 2: Qwen2.5-1.5B-shaped cache: prefill, appends, full-prefix decode -------------

def test_config2_qwen_shaped_prefill_append_decode():
    shp = wl.QWEN25_1P5B
    D, T0, steps = shp.head_dim, shp.prefix, 128      # the configuration's 128 decode steps
    S = shp.streams  # 112 streams: (layer, K/V, head)
    T_max = T0 + steps
    per_lambda = shp.kv_heads  # one lambda row per (layer, K/V): 56 rows
    n_lambda = S // per_lambda
    plan = kb.Plan(D, G, 77)
    sg = plan.signs()
    lam = wl.make_lambda(n_lambda, D, 21)
    # stream i is K-like for even (layer, kv) index, V-like for odd
    xs = []
    for i in range(n_lambda):
        kind = "k_outlier" if i % 2 == 0 else "gaussian"
        xs.append(wl.make_vectors(per_lambda * T_max, D, shp.dtype, kind, 500 + i).view(per_lambda, T_max, D))
    x_all = torch.cat(xs, 0)  # [S, T_max, D]
    lamd = lam.cuda()
    packed = torch.zeros(S, T_max, D // 2, dtype=torch.uint8, device="cuda")
    scales = torch.zeros(S, T_max, D // G, dtype=torch.float16, device="cuda")
    # prefill: one encode per stream block sharing a lambda row (rows of a stream are contiguous in the cache)
    for i in range(n_lambda):
        for h in range(per_lambda):
            s = i * per_lambda + h
            xp = x_all[s, :T0].contiguous().cuda()
            kb.kvq_encode(plan.handle, xp, lamd[i], packed[s, :T0], scales[s, :T0])
    # decode steps: append one vector per stream
    for t in range(steps):
        xn = x_all[:, T0 + t].contiguous().cuda()
        kb.kvq_append(plan.handle, xn, lamd, packed, scales, T0 + t, per_lambda)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    # oracle on the whole cache [S*T_max rows, lambda row = stream // per_lambda]
    ora = ko.encode(bits(x_all.reshape(-1, D)), ko.F16, sg, lam.numpy(), G, per_lambda * T_max, want_v=True)
    parity.check_encode(packed.view(-1, D // 2).cpu().numpy(), bits(scales.view(-1, D // G)), ora, G, "qwen cache")
    # full-prefix decode of the whole cache in one launch
    out = gpu_decode(plan, packed.view(-1, D // 2), scales.view(-1, D // G), lamd, shp.dtype, per_lambda * T_max)
    ob, o64 = ko.decode(packed.view(-1, D // 2).cpu().numpy(), bits(scales.view(-1, D // G)), sg, lam.numpy(), G,
                        ko.F16, per_lambda * T_max, want_f64=True)
    parity.check_decode(bits(out), ob, o64, ko.F16, "qwen full-prefix decode")
    plan.close()


def test_append_touches_only_row_pos():
    D, S, T = 128, 37, 9
    plan = kb.Plan(D, G, 5)
    x = wl.make_vectors(S, D, "f16", "gaussian", 9).cuda()
    lam = wl.make_lambda(S, D, 10).cuda()
    packed = torch.full((S, T, D // 2), 0xAB, dtype=torch.uint8, device="cuda")
    scales = torch.full((S, T, D // G), 1.25, dtype=torch.float16, device="cuda")
    kb.kvq_append(plan.handle, x, lam, packed, scales, 4, 1)
    torch.cuda.synchronize()
    keep = [t for t in range(T) if t != 4]
    assert bool((packed[:, keep] == 0xAB).all()) and bool((scales[:, keep] == 1.25).all())
    # the oracle's append leaves the same rows alone and writes, at row 4, what its encode of the 37 vectors gives
    pc = np.full((S, T, D // 2), 0xAB, dtype=np.uint8)
    sc = np.full((S, T, D // G), np.float16(1.25).view(np.uint16), dtype=np.uint16)
    ko.append(bits(x), ko.F16, plan.signs(), lam.cpu().numpy(), G, pc, sc, 4, 1)
    assert (pc[:, keep] == 0xAB).all() and (sc[:, keep] == np.float16(1.25).view(np.uint16)).all()
    ora = ko.encode(bits(x), ko.F16, plan.signs(), lam.cpu().numpy(), G, 1, want_v=True)
    assert np.array_equal(pc[:, 4], ora["packed"]) and np.array_equal(sc[:, 4], ora["scales"])
    # and the library's row 4 against it, under the code, tie and scale rules (4736 codes: one mismatch at a tie would
    # already be 2e-4 of them, so the share rule of the sampled tests applies; in practice they are identical)
    enc = parity.check_encode(packed[:, 4].contiguous().cpu().numpy(), bits(scales[:, 4].contiguous()), ora, G, "append row", min_agree=0.9995)
    assert enc["mismatches"] <= 1
    plan.close()


@pytest.mark.parametrize("D,dtype,S,T_max,spl,blocks", [
    (128, "f16", 112, 300, 2, (256, 1, 16, 27)),       # a prefill block, then window flushes of 1, 16 and a ragged 27
    (128, "f16", 3, 9000, 1, (8192, 64)),              # blocks long enough for the tensor-core encode
    (256, "bf16", 26, 80, 1, (33, 32, 15)),
    (96, "f16", 7, 40, 7, (5, 35)),
    # blocks of 64 rows and more on plans without a rotation: the tensor-core decode reads and writes the window of every
    # stream's cache in place (tiles that end inside a stream's window, lambda rows shared by several streams, a window
    # that starts past row 0)
    (256, "bf16", 20, 400, 3, (200, 130, 70)),
    (160, "f16", 9, 500, 2, (300, 129)),
    (64, "bf16", 40, 200, 5, (128, 65)),
    (128, "bf16", 33, 260, 4, (64, 196)),
])
def test_flush_block_fills_the_int4_and_the_dequantized_caches(D, dtype, S, T_max, spl, blocks):
    odt = ko.F16 if dtype == "f16" else ko.BF16
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    plan = kb.Plan(D, G, 31)
    sg = plan.signs()
    n_lambda = (S + spl - 1) // spl
    lam = wl.make_lambda(n_lambda, D, 61)
    x_all = wl.make_vectors(S * T_max, D, dtype, "k_outlier", 62).view(S, T_max, D)
    packed = torch.full((S, T_max, D // 2), 0xAB, dtype=torch.uint8, device="cuda")
    scales = torch.full((S, T_max, D // G), 1.25, dtype=torch.float16, device="cuda")
    dq = torch.full((S, T_max, D), 3.0, dtype=tdt, device="cuda")
    lamd = lam.cuda()
    pos = 0
    for rows in blocks:
        kb.kvq_flush_block(plan.handle, x_all[:, pos:pos + rows].contiguous().cuda(), lamd, packed, scales, dq, pos, spl)
        pos += rows
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    # rows past the flushed prefix are untouched
    assert bool((packed[:, pos:] == 0xAB).all()) and bool((scales[:, pos:] == 1.25).all()) and bool((dq[:, pos:] == 3.0).all())
    # the int4 cache equals one encode of the whole prefix (oracle), the dequantized cache its full-prefix decode
    xp = x_all[:, :pos].reshape(-1, D)
    ora = ko.encode(bits(xp), odt, sg, lam.numpy(), G, spl * pos, want_v=True)
    pk = packed[:, :pos].reshape(-1, D // 2).cpu().numpy()
    sb = bits(scales[:, :pos].reshape(-1, D // G))
    parity.check_encode(pk, sb, ora, G, "flush int4 cache")
    ob, o64 = ko.decode(pk, sb, sg, lam.numpy(), G, odt, spl * pos, want_f64=True)
    parity.check_decode(bits(dq[:, :pos].reshape(-1, D)), ob, o64, odt, "flush dequantized cache")
    # and the product's own full-prefix decode of the int4 cache gives the same rows (the incremental path's claim)
    full = gpu_decode(plan, packed[:, :pos].reshape(-1, D // 2).contiguous(), scales[:, :pos].reshape(-1, D // G).contiguous(),
                      lamd, dtype, spl * pos)
    parity.check_decode(bits(full), ob, o64, odt, "full-prefix decode of the flushed cache")
    plan.close()


@pytest.mark.parametrize("D", [64, 96, 128, 160, 256])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("group,nbits", [(G, 4), (0, 4), (G, 8)])
def test_window_flush_in_one_launch_equals_decode_of_what_it_stored(D, dtype, group, nbits):
    """A small flush runs as ONE matrix-vector launch that dequantizes in the encode's registers; the rows it leaves in the
    dequantized cache must be, bit for bit, what the matrix-vector kvq_decode makes of the codes and scales it stored."""
    g = group or D
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    S, T_max, rows, pos0, spl = 13, 40, 11, 17, 3        # 143 vectors: 17 full CTAs of 8 and a ragged one
    plan = kb.Plan(D, g, 77, nbits)
    lamd = wl.make_lambda((S + spl - 1) // spl, D, 78).cuda()
    x = wl.make_vectors(S * rows, D, dtype, "k_outlier", 79).view(S, rows, D).cuda()
    packed = torch.full((S, T_max, D * nbits // 8), 0xAB, dtype=torch.uint8, device="cuda")
    scales = torch.full((S, T_max, D // g), 1.25, dtype=torch.float16, device="cuda")
    dq = torch.full((S, T_max, D), 3.0, dtype=tdt, device="cuda")
    n0 = kb.kvq_launch_count()
    kb.kvq_flush_block(plan.handle, x, lamd, packed, scales, dq, pos0, spl)
    assert kb.kvq_launch_count() - n0 == 1
    # the caches hold what the two-launch form (append-style encode, then decode) stores
    p2, s2 = torch.full_like(packed, 0xAB), torch.full_like(scales, 1.25)
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_MATVEC, kb.KVQ_IMPL_FFT)   # a decode side that is not matrix-vector: two launches
    dq2 = torch.full_like(dq, 3.0)
    n0 = kb.kvq_launch_count()
    kb.kvq_flush_block(plan.handle, x, lamd, p2, s2, dq2, pos0, spl)
    assert kb.kvq_launch_count() - n0 == 2
    assert torch.equal(packed, p2) and torch.equal(scales, s2)
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_MATVEC, kb.KVQ_IMPL_MATVEC)
    blk_p = packed[:, pos0:pos0 + rows].reshape(S * rows, -1).contiguous()
    blk_s = scales[:, pos0:pos0 + rows].reshape(S * rows, -1).contiguous()
    out = torch.empty(S * rows, D, dtype=tdt, device="cuda")
    kb.kvq_decode(plan.handle, blk_p, blk_s, lamd, out, spl * rows)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    assert torch.equal(dq[:, pos0:pos0 + rows].reshape(S * rows, D).view(torch.int16), out.view(torch.int16))
    mask = torch.ones(T_max, dtype=torch.bool, device="cuda")
    mask[pos0:pos0 + rows] = False
    assert bool((dq[:, mask] == 3.0).all()) and bool((packed[:, mask] == 0xAB).all()) and bool((scales[:, mask] == 1.25).all())
    plan.close()


# ---- the cache position in device memory: kvq_append_at / kvq_flush_block_at, eager and replayed from a CUDA graph ----

@pytest.mark.parametrize("D,dtype,group,nbits", [(128, "f16", G, 4), (256, "bf16", G, 4), (96, "f16", G, 4), (160, "bf16", G, 4),
                                                 (64, "f16", 0, 4), (128, "bf16", G, 8)])
def test_position_in_device_memory_gives_what_the_host_position_gives(D, dtype, group, nbits):
    g = group or D
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    S, T_max, rows, spl = 21, 48, 5, 4
    plan = kb.Plan(D, g, 91, nbits)
    lamd = wl.make_lambda((S + spl - 1) // spl, D, 92).cuda()
    x_new = wl.make_vectors(S * 3, D, dtype, "k_outlier", 93).view(3, S, D).cuda()
    x_blk = wl.make_vectors(S * rows * 2, D, dtype, "k_outlier", 94).view(2, S, rows, D).cuda()

    def caches():
        return (torch.full((S, T_max, D * nbits // 8), 0xAB, dtype=torch.uint8, device="cuda"),
                torch.full((S, T_max, D // g), 1.25, dtype=torch.float16, device="cuda"),
                torch.full((S, T_max, D), 3.0, dtype=tdt, device="cuda"))

    pa, sa, da = caches()       # positions from the host
    pb, sb, db = caches()       # the same positions from device memory
    pos = torch.zeros(1, dtype=torch.int64, device="cuda")
    steps = [("append", 0, 0), ("append", 1, T_max - 1), ("flush", 0, 7), ("append", 2, 12), ("flush", 1, T_max - rows)]
    for kind, i, p in steps:
        pos.fill_(p)
        if kind == "append":
            kb.kvq_append(plan.handle, x_new[i], lamd, pa, sa, p, spl)
            kb.kvq_append_at(plan.handle, x_new[i], lamd, pb, sb, pos, spl)
        else:
            kb.kvq_flush_block(plan.handle, x_blk[i], lamd, pa, sa, da, p, spl)
            kb.kvq_flush_block_at(plan.handle, x_blk[i], lamd, pb, sb, db, pos, spl)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    assert torch.equal(pa, pb) and torch.equal(sa, sb) and torch.equal(da.view(torch.int16), db.view(torch.int16))
    assert not bool((pa[:, 7:7 + rows] == 0xAB).all())      # something was written at all

    # a position outside the cache: nothing is written, the plan's status word says so, and clearing it restores service
    for bad, call in ((T_max, "append"), (-1, "append"), (T_max - rows + 1, "flush"), (-3, "flush")):
        pos.fill_(bad)
        if call == "append":
            kb.kvq_append_at(plan.handle, x_new[0], lamd, pb, sb, pos, spl)
        else:
            kb.kvq_flush_block_at(plan.handle, x_blk[0], lamd, pb, sb, db, pos, spl)
        assert kb.kvq_plan_device_status(plan.handle) == kb.KVQ_DEV_POSITION
        assert torch.equal(pa, pb) and torch.equal(sa, sb) and torch.equal(da.view(torch.int16), db.view(torch.int16))
        kb.kvq_plan_clear_device_status(plan.handle)
        assert kb.kvq_plan_device_status(plan.handle) == 0
    plan.close()


def test_append_at_beyond_the_small_call_limit_against_the_oracle():
    """kvq_append_at always takes the matrix-vector kernel: 5120 streams (every layer, head and sequence of a large model in
    one call) is past the size where kvq_append would change kernels."""
    D, S, T_max, spl = 128, 5120, 6, 64
    plan = kb.Plan(D, G, 95)
    sg = plan.signs()
    lam = wl.make_lambda(S // spl, D, 96)
    x = wl.make_vectors(S, D, "f16", "k_outlier", 97)
    packed = torch.full((S, T_max, D // 2), 0xAB, dtype=torch.uint8, device="cuda")
    scales = torch.full((S, T_max, D // G), 1.25, dtype=torch.float16, device="cuda")
    pos = torch.full((1,), 4, dtype=torch.int64, device="cuda")
    n0 = kb.kvq_launch_count()
    kb.kvq_append_at(plan.handle, x.cuda(), lam.cuda(), packed, scales, pos, spl)
    assert kb.kvq_launch_count() - n0 == 1
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    ora = ko.encode(bits(x), ko.F16, sg, lam.numpy(), G, spl, want_v=True)
    parity.check_encode(packed[:, 4].contiguous().cpu().numpy(), bits(scales[:, 4].contiguous()), ora, G, "append_at, 5120 streams")
    keep = [0, 1, 2, 3, 5]
    assert bool((packed[:, keep] == 0xAB).all()) and bool((scales[:, keep] == 1.25).all())
    plan.close()


@pytest.mark.parametrize("D,dtype", [(64, "bf16"), (96, "f16"), (128, "f16"), (128, "bf16")])
def test_matvec_kernels_past_one_resident_wave(D, dtype):
    """More batches of 8 vectors than the device holds CTAs: a CTA of the D <= 128 kernels then takes several batches with its
    table slice kept in registers.  Encode and decode against the oracle; the fused flush against the two-launch flush."""
    run_case(D, dtype, 6007, "k_outlier", 7300 + D, n_lambda=3, rows_per_lambda=2100, enc_impl="matvec", dec_impl="matvec")
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    S, T_max, rows, spl = 150, 40, 33, 50          # 4950 vectors: 619 batches
    plan = kb.Plan(D, G, 7400 + D)
    lamd = wl.make_lambda(S // spl, D, 7401).cuda()
    x = wl.make_vectors(S * rows, D, dtype, "k_outlier", 7402).view(S, rows, D).cuda()
    pos0 = torch.full((1,), 5, dtype=torch.int64, device="cuda")
    pa = torch.zeros(S, T_max, D // 2, dtype=torch.uint8, device="cuda")
    sa = torch.zeros(S, T_max, D // G, dtype=torch.float16, device="cuda")
    da = torch.zeros(S, T_max, D, dtype=tdt, device="cuda")
    pb, sb, db = torch.zeros_like(pa), torch.zeros_like(sa), torch.zeros_like(da)
    n0 = kb.kvq_launch_count()
    kb.kvq_flush_block_at(plan.handle, x, lamd, pa, sa, da, pos0, spl)              # one fused launch, looping CTAs
    assert kb.kvq_launch_count() - n0 == 1
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_MATVEC, kb.KVQ_IMPL_MATVEC)
    kb.kvq_append(plan.handle, x[:, 0].contiguous(), lamd, pb, sb, 5, spl)           # the same rows by the unfused calls
    for i in range(1, rows):
        kb.kvq_append(plan.handle, x[:, i].contiguous(), lamd, pb, sb, 5 + i, spl)
    blk_p = pb[:, 5:5 + rows].reshape(S * rows, -1).contiguous()
    blk_s = sb[:, 5:5 + rows].reshape(S * rows, -1).contiguous()
    out = torch.empty(S * rows, D, dtype=tdt, device="cuda")
    kb.kvq_decode(plan.handle, blk_p, blk_s, lamd, out, spl * rows)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    assert torch.equal(pa, pb) and torch.equal(sa, sb)
    assert torch.equal(da[:, 5:5 + rows].reshape(S * rows, D).view(torch.int16), out.view(torch.int16))
    assert bool((da[:, :5] == 0).all()) and bool((da[:, 5 + rows:] == 0).all())
    plan.close()


def test_decode_loop_replayed_from_a_cuda_graph():
    """One decode step of the cache side -- advance the position word, append the new token of every stream, and flush the
    window when it is full -- recorded once and replayed: the caches equal those of the same steps issued call by call."""
    D, S, T_max, W, spl = 128, 16, 64, 4, 8
    plan = kb.Plan(D, G, 98)
    lamd = wl.make_lambda(S // spl, D, 99).cuda()
    n_steps = 3 * W
    xs = wl.make_vectors(n_steps * S, D, "f16", "k_outlier", 100).view(n_steps, S, D).cuda()

    def caches():
        return (torch.zeros(S, T_max, D // 2, dtype=torch.uint8, device="cuda"),
                torch.zeros(S, T_max, D // G, dtype=torch.float16, device="cuda"),
                torch.zeros(S, T_max, D, dtype=torch.float16, device="cuda"))

    # reference: call by call with host positions
    pa, sa, da = caches()
    for t in range(n_steps):
        kb.kvq_append(plan.handle, xs[t], lamd, pa, sa, t, spl)
        if (t + 1) % W == 0:
            blk = xs[t + 1 - W:t + 1].transpose(0, 1).contiguous()
            kb.kvq_flush_block(plan.handle, blk, lamd, pa, sa, da, t + 1 - W, spl)
    torch.cuda.synchronize()

    # graphs: static inputs, the positions in device memory.  Two graphs, as a serving loop would hold: the every-step one
    # and the one for steps that end a window.
    pb, sb, db = caches()
    x_static = torch.zeros(S, D, dtype=torch.float16, device="cuda")
    blk_static = torch.zeros(S, W, D, dtype=torch.float16, device="cuda")
    pos = torch.zeros(1, dtype=torch.int64, device="cuda")
    pos0 = torch.zeros(1, dtype=torch.int64, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):      # the plan's first use on the device and the kernels' first launches happen here
        kb.kvq_append_at(plan.handle, x_static, lamd, pb, sb, pos, spl)
        kb.kvq_flush_block_at(plan.handle, blk_static, lamd, pb, sb, db, pos0, spl)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    pb.zero_(), sb.zero_(), db.zero_()
    g_step, g_flush = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
    with torch.cuda.graph(g_step):
        kb.kvq_append_at(plan.handle, x_static, lamd, pb, sb, pos, spl)
        pos.add_(1)
    with torch.cuda.graph(g_flush):
        kb.kvq_flush_block_at(plan.handle, blk_static, lamd, pb, sb, db, pos0, spl)
        pos0.add_(W)
    pb.zero_(), sb.zero_(), db.zero_(), pos.zero_(), pos0.zero_()
    for t in range(n_steps):
        x_static.copy_(xs[t])
        g_step.replay()
        if (t + 1) % W == 0:
            blk_static.copy_(xs[t + 1 - W:t + 1].transpose(0, 1))
            g_flush.replay()
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    assert int(pos.item()) == n_steps and int(pos0.item()) == n_steps
    assert torch.equal(pa, pb) and torch.equal(sa, sb) and torch.equal(da.view(torch.int16), db.view(torch.int16))
    assert bool((pb[:, :n_steps] != 0).any())
    plan.close()


def test_flush_block_rejects_blocks_outside_the_cache():
    D, S, T = 128, 4, 16
    plan = kb.Plan(D, G, 1)
    x = wl.make_vectors(S * 8, D, "f16", "gaussian", 1).view(S, 8, D).cuda()
    lam = wl.make_lambda(1, D, 2).cuda()
    packed = torch.zeros(S, T, D // 2, dtype=torch.uint8, device="cuda")
    scales = torch.zeros(S, T, D // G, dtype=torch.float16, device="cuda")
    dq = torch.zeros(S, T, D, dtype=torch.float16, device="cuda")
    with pytest.raises(kb.KvqError):
        kb.kvq_flush_block(plan.handle, x, lam, packed, scales, dq, 9, 0)
    with pytest.raises(kb.KvqError):
        kb.kvq_flush_block(plan.handle, x, lam, packed, scales, dq, -1, 0)
    kb.kvq_flush_block(plan.handle, x, lam, packed, scales, dq, 8, 0)     # the last block that fits
    kb.kvq_flush_block(plan.handle, x[:, :0], lam, packed, scales, dq, 16, 0)   # an empty block is a no-op
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    plan.close()


# ---- the matrix-vector kernels of the small calls, forced at sizes that span many CTAs and a ragged last one ------

@pytest.mark.parametrize("D,dtype", [(64, "f16"), (64, "bf16"), (96, "f16"), (96, "bf16"), (128, "f16"), (128, "bf16"),
                                     (160, "f16"), (160, "bf16"), (256, "f16"), (256, "bf16")])
def test_matvec_kernels_all_dims(D, dtype):
    run_case(D, dtype, 2051, "k_outlier", 7000 + D, n_lambda=5, rows_per_lambda=411, enc_impl="matvec", dec_impl="matvec")
    run_case(D, dtype, 5, "gaussian", 7100 + D, enc_impl="matvec", dec_impl="matvec")


def test_small_calls_take_the_matvec_kernels_and_agree_with_the_fft():
    # AUTO below 2048 rows is the matrix-vector kernel; its codes agree with the register FFT except at rounding ties
    D, N = 128, 1500
    plan = kb.Plan(D, G, 11)
    x = wl.make_vectors(N, D, "f16", "k_outlier", 12).cuda()
    lam = wl.make_lambda(1, D, 13).cuda()
    n0 = kb.kvq_launch_count()
    pa, sa = gpu_encode(plan, x, lam)
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_MATVEC, kb.KVQ_IMPL_MATVEC)
    pm, sm_ = gpu_encode(plan, x, lam)
    assert torch.equal(pa, pm) and torch.equal(sa, sm_)
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_FFT, kb.KVQ_IMPL_FFT)
    pf, sf = gpu_encode(plan, x, lam)
    assert kb.kvq_launch_count() - n0 == 3
    assert float((pa == pf).float().mean()) > 0.999 and float((sa == sf).float().mean()) > 0.99
    plan.close()


# ---- base variants: one scale per vector and / or 8-bit codes (register-FFT kernels) -------------------

@pytest.mark.parametrize("D,dtype,per_vector,nbits", [
    (64, "f16", True, 4), (64, "f16", True, 8), (64, "bf16", False, 8),
    (96, "f16", True, 4), (96, "bf16", True, 8),
    (128, "f16", True, 4), (128, "f16", False, 8), (128, "bf16", True, 8),
    (160, "f16", True, 8), (160, "bf16", False, 8),
    (256, "bf16", True, 4), (256, "f16", True, 8), (256, "bf16", False, 8),
])
@pytest.mark.parametrize("impl", ["fft", "matvec", "gemm"])
def test_base_variants_per_vector_scale_and_byte_codes(D, dtype, per_vector, nbits, impl):
    if impl == "gemm" and D == 160 and dtype == "bf16":
        pytest.skip("no tensor-core kernel for this layout: covered by the refusal test")
    # byte codes at D = 256: the tensor cores decode them and encode them from fp16; from bf16 the encode stays on the register FFT
    enc_impl = "fft" if impl == "gemm" and D == 256 and nbits == 8 and dtype == "bf16" else impl
    N, n_lambda, rpl = 5003, 3, 1700          # ragged, lambda rows straddle the warps' tiles
    group = D if per_vector else G
    odt = ko.F16 if dtype == "f16" else ko.BF16
    plan = kb.Plan(D, group, 90 + D, bits=nbits)
    kb.kvq_plan_set_impl(plan.handle, IMPL[enc_impl], IMPL[impl])
    sg = plan.signs()
    lam = wl.make_lambda(n_lambda, D, 91)
    x = wl.make_vectors(N, D, dtype, "k_outlier", 92 + nbits)
    xd, lamd = x.cuda(), lam.cuda()
    packed, scales = plan.empty_packed(N), plan.empty_scales(N)
    assert packed.shape == (N, D * nbits // 8) and scales.shape == (N, D // group)
    kb.kvq_encode(plan.handle, xd, lamd, packed, scales, rpl)
    out = torch.empty(N, D, dtype=xd.dtype, device="cuda")
    kb.kvq_decode(plan.handle, packed, scales, lamd, out, rpl)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    ora = ko.encode(bits(x), odt, sg, lam.numpy(), group, rpl, want_v=True, bits=nbits)
    pk, sb = packed.cpu().numpy(), bits(scales)
    parity.check_encode(pk, sb, ora, group, "variant encode", bits=nbits)
    ob, o64 = ko.decode(pk, sb, sg, lam.numpy(), group, odt, rpl, want_f64=True, bits=nbits)
    parity.check_decode(bits(out), ob, o64, odt, "variant decode")
    plan.close()


@pytest.mark.parametrize("dtype,per_vector", [("f16", False), ("bf16", False), ("bf16", True)])
def test_byte_codes_at_d256_decode_on_the_tensor_cores(dtype, per_vector):
    """8-bit codes (Sec. 3.2 step 4's int8 output) at D = 256 through the radix-2 tensor-core decode: rows of 256 bytes loaded
    as two boxes, bytes routed by channel parity; several CTAs, lambda rows that end inside tiles, AUTO and forced."""
    D, N, n_lambda, rpl = 256, 21000, 5, 4300
    group = D if per_vector else G
    odt = DT[dtype]
    plan = kb.Plan(D, group, 300, bits=8)
    sg = plan.signs()
    lam = wl.make_lambda(n_lambda, D, 301)
    x = wl.make_vectors(N, D, dtype, "k_outlier", 302)
    ora = ko.encode(bits(x), odt, sg, lam.numpy(), group, rpl, want_v=True, bits=8)
    ob, o64 = ko.decode(ora["packed"], ora["scales"], sg, lam.numpy(), group, odt, rpl, want_f64=True, bits=8)
    pk = torch.from_numpy(ora["packed"]).cuda()
    sc = torch.from_numpy(ora["scales"].view(np.int16)).view(torch.float16).cuda()
    for impl in (kb.KVQ_IMPL_GEMM, kb.KVQ_IMPL_AUTO):
        kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_AUTO, impl)
        n0 = kb.kvq_launch_count()
        out = gpu_decode_raw(plan, pk, sc, lam.cuda(), dtype, rpl)
        assert kb.kvq_launch_count() - n0 == 1
        parity.check_decode(bits(out), ob, o64, odt, "byte codes, D = 256, tensor-core decode")
    if dtype == "f16":   # the tensor-core encode takes byte codes from fp16 input (two fp16 terms of W carry 22 bits)
        kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_GEMM, kb.KVQ_IMPL_AUTO)
        packed, scales = gpu_encode(plan, x.cuda(), lam.cuda(), rpl)
        parity.check_encode(packed.cpu().numpy(), bits(scales), ora, group, "byte codes, D = 256, tensor-core encode", bits=8)
    plan.close()


@pytest.mark.parametrize("D,dtype,N,n_lambda,rpl", [
    (128, "f16", 20000, 1, 0), (128, "f16", 40000, 200, 200), (128, "bf16", 20000, 3, 7000), (64, "f16", 9000, 1, 0),
    (64, "bf16", 9000, 2, 4500), (96, "f16", 9000, 1, 0), (96, "bf16", 5000, 1, 0), (160, "f16", 9000, 4, 2300),
    (160, "bf16", 9000, 2, 4600), (256, "f16", 9000, 1, 0), (256, "bf16", 9000, 3, 3100), (256, "bf16", 60000, 300, 200), (256, "f16", 129, 1, 0),
])
def test_one_scale_per_vector_on_the_tensor_cores(D, dtype, N, n_lambda, rpl):
    # group = D, 4-bit codes: the tensor-core encode trades the row maximum between its two half-row threads (D <= 160)
    # or between the four of a cluster pair (D = 256), the tensor-core decode reads one scale per row
    odt = ko.F16 if dtype == "f16" else ko.BF16
    plan = kb.Plan(D, D, 60 + D)
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_GEMM, kb.KVQ_IMPL_GEMM)
    sg = plan.signs()
    lam = wl.make_lambda(n_lambda, D, 61)
    x = wl.make_vectors(N, D, dtype, "k_outlier", 62 + N)
    packed, scales = gpu_encode(plan, x.cuda(), lam.cuda(), rpl)
    assert scales.shape == (N, 1)
    ora = ko.encode(bits(x), odt, sg, lam.numpy(), D, rpl, want_v=True)
    pk, sb = packed.cpu().numpy(), bits(scales)
    parity.check_encode(pk, sb, ora, D, "per-vector encode")
    out = gpu_decode(plan, packed, scales, lam.cuda(), dtype, rpl)
    ob, o64 = ko.decode(pk, sb, sg, lam.numpy(), D, odt, rpl, want_f64=True)
    parity.check_decode(bits(out), ob, o64, odt, "per-vector decode")
    plan.close()


def test_base_variants_append_and_flush_and_refusals():
    D, S, T = 256, 24, 40
    plan = kb.Plan(D, D, 7, bits=8)
    sg = plan.signs()
    lam = wl.make_lambda(S, D, 8)
    x = wl.make_vectors(S * T, D, "f16", "gaussian", 9).view(S, T, D)   # byte codes at D = 256: register FFT and matrix-vector only
    packed = torch.full((S, T, D), 0x55, dtype=torch.uint8, device="cuda")
    scales = torch.full((S, T, 1), 2.0, dtype=torch.float16, device="cuda")
    dq = torch.full((S, T, D), 3.0, dtype=torch.float16, device="cuda")
    lamd = lam.cuda()
    kb.kvq_flush_block(plan.handle, x[:, :32].contiguous().cuda(), lamd, packed, scales, dq, 0, 1)
    for t in range(32, 37):
        kb.kvq_append(plan.handle, x[:, t].contiguous().cuda(), lamd, packed, scales, t, 1)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    assert bool((packed[:, 37:] == 0x55).all()) and bool((scales[:, 37:] == 2.0).all()) and bool((dq[:, 32:] == 3.0).all())
    ora = ko.encode(bits(x[:, :37].reshape(-1, D)), ko.F16, sg, lam.numpy(), D, 37, want_v=True, bits=8)
    pk, sb = packed[:, :37].reshape(-1, D).cpu().numpy(), bits(scales[:, :37].reshape(-1, 1))
    parity.check_encode(pk, sb, ora, D, "variant cache", bits=8)
    pk32, sb32 = packed[:, :32].reshape(-1, D).cpu().numpy(), bits(scales[:, :32].reshape(-1, 1))
    ob, o64 = ko.decode(pk32, sb32, sg, lam.numpy(), D, ko.F16, 32, want_f64=True, bits=8)
    parity.check_decode(bits(dq[:, :32].reshape(-1, D)), ob, o64, ko.F16, "variant dequantized cache")
    # byte codes at D = 256: the tensor cores decode them (the flushed rows: the same values as the dequantized cache up to
    # the families' rounding), but have no encode for them
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_GEMM, kb.KVQ_IMPL_GEMM)
    o = torch.empty(S * 32, D, dtype=torch.float16, device="cuda")
    kb.kvq_decode(plan.handle, packed[:, :32].reshape(-1, D).contiguous(), scales[:, :32].reshape(-1, 1).contiguous(), lamd, o, 32)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    parity.check_decode(bits(o), ob, o64, ko.F16, "variant cache, tensor-core decode")
    # ... and encode them from fp16 (the whole cache again, as one flat call), but not from bf16
    p2, s2 = torch.empty(S * T, D, dtype=torch.uint8, device="cuda"), torch.empty(S * T, 1, dtype=torch.float16, device="cuda")
    kb.kvq_encode(plan.handle, x.reshape(-1, D).cuda(), lamd, p2, s2, T)
    torch.cuda.synchronize()
    assert kb.kvq_plan_device_status(plan.handle) == 0
    ora_all = ko.encode(bits(x.reshape(-1, D)), ko.F16, sg, lam.numpy(), D, T, want_v=True, bits=8)
    parity.check_encode(p2.cpu().numpy(), bits(s2), ora_all, D, "byte codes, D = 256, tensor-core encode", bits=8, min_agree=0.9995)
    with pytest.raises(kb.KvqError):
        kb.kvq_encode(plan.handle, x.reshape(-1, D).to(torch.bfloat16).cuda(), lamd, packed.view(-1, D), scales.view(-1, 1), T)
    plan.close()
    with pytest.raises(kb.KvqError):
        kb.Plan(128, 64, 1)           # groups other than 32 or D
    with pytest.raises(kb.KvqError):
        kb.Plan(128, 32, 1, bits=6)


# ---- rotation between the transform and lambda, folded into the tensor-core kernels' tables ---------------

@pytest.mark.parametrize("D,dtype,near", [
    (64, "f16", 0.0), (96, "f16", 0.02), (128, "f16", 0.0), (128, "f16", 0.02), (160, "f16", 0.0),
    (256, "f16", 0.0), (256, "bf16", 0.0), (256, "bf16", 0.02),
])
def test_rotated_plan_matches_the_oracle(D, dtype, near):
    N, n_lambda, rpl = 3000, 3, 1100           # ragged; lambda rows end inside tiles
    odt = ko.F16 if dtype == "f16" else ko.BF16
    plan = kb.Plan(D, G, 300 + D)
    sg = plan.signs()
    R = wl.make_rotation(D, 301, near)
    plan.set_rotation(R)
    Rd = R.numpy().astype(np.float64)
    lam = wl.make_lambda(n_lambda, D, 302)
    x = wl.make_vectors(N, D, dtype, "k_outlier", 303)
    packed, scales = gpu_encode(plan, x.cuda(), lam.cuda(), rpl)
    ora = ko.encode(bits(x), odt, sg, lam.numpy(), G, rpl, want_v=True, rot=Rd)
    pk, sb = packed.cpu().numpy(), bits(scales)
    parity.check_encode(pk, sb, ora, G, "rotated encode")
    out = gpu_decode(plan, packed, scales, lam.cuda(), dtype, rpl)
    ob, o64 = ko.decode(pk, sb, sg, lam.numpy(), G, odt, rpl, want_f64=True, rot=Rd)
    parity.check_decode(bits(out), ob, o64, odt, "rotated decode")
    # the rotation matters: without it the oracle gives other codes
    assert (ko.encode(bits(x[:64]), odt, sg, lam.numpy()[:1], G)["codes"] != ora["codes"][:64]).mean() > 0.2
    plan.close()


def test_rotation_can_be_set_and_removed_on_a_plan_in_use():
    D, N = 128, 2048
    plan = kb.Plan(D, G, 5)
    sg = plan.signs()
    lam = wl.make_lambda(1, D, 6)
    x = wl.make_vectors(N, D, "f16", "gaussian", 7)
    xd, lamd = x.cuda(), lam.cuda()
    base = [t.clone() for t in gpu_encode(plan, xd, lamd)]            # first use: the device tables now exist
    R = wl.make_rotation(D, 8)
    plan.set_rotation(R)                                               # rewrites them in place
    packed, scales = gpu_encode(plan, xd, lamd)                        # small call: still the tensor-core path
    ora = ko.encode(bits(x), ko.F16, sg, lam.numpy(), G, want_v=True, rot=R.numpy().astype(np.float64))
    parity.check_encode(packed.cpu().numpy(), bits(scales), ora, G, "rotation set after first use")
    # append on a rotated plan
    pc = torch.zeros(N, 4, D // 2, dtype=torch.uint8, device="cuda")
    sc = torch.zeros(N, 4, D // G, dtype=torch.float16, device="cuda")
    kb.kvq_append(plan.handle, xd, lamd, pc, sc, 2, 0)
    torch.cuda.synchronize()
    parity.check_encode(pc[:, 2].contiguous().cpu().numpy(), bits(sc[:, 2].contiguous()), ora, G, "rotated append")
    assert bool((pc[:, [0, 1, 3]] == 0).all())
    # calibration sees the rotated coordinates
    lam_cal = torch.empty(D, dtype=torch.float32, device="cuda")
    kb.kvq_calibrate_lambda(plan.handle, xd, lam_cal)
    torch.cuda.synchronize()
    v1 = ko.encode(bits(x), ko.F16, sg, np.ones(D, np.float32), G, want_v=True, rot=R.numpy().astype(np.float64))["v"]
    amax = np.abs(v1).max(axis=0)
    assert np.abs(1.0 / lam_cal.cpu().numpy().astype(np.float64) - amax).max() <= 2e-6 * np.linalg.norm(v1, axis=1).max()
    # the window flush of a rotated plan (matrix-vector kernels)
    dq = torch.zeros(N, 4, D, dtype=torch.float16, device="cuda")
    kb.kvq_flush_block(plan.handle, xd.view(N, 1, D), lamd, pc, sc, dq, 1, 0)
    torch.cuda.synchronize()
    pk1, sb1 = pc[:, 1].contiguous().cpu().numpy(), bits(sc[:, 1].contiguous())
    parity.check_encode(pk1, sb1, ora, G, "rotated flush")
    ob, o64 = ko.decode(pk1, sb1, sg, lam.numpy(), G, ko.F16, want_f64=True, rot=R.numpy().astype(np.float64))
    parity.check_decode(bits(dq[:, 1].contiguous()), ob, o64, ko.F16, "rotated flush, dequantized rows")
    # what a rotated plan refuses: the register FFT
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_FFT, kb.KVQ_IMPL_FFT)
    with pytest.raises(kb.KvqError):
        gpu_encode(plan, xd, lamd)
    with pytest.raises(kb.KvqError):
        kb.kvq_decode(plan.handle, packed, scales, lamd, torch.empty(N, D, dtype=torch.float16, device="cuda"), 0)
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_AUTO, kb.KVQ_IMPL_AUTO)
    # and removed again: the plan is what it was
    plan.set_rotation(None)
    again = gpu_encode(plan, xd, lamd)
    assert torch.equal(again[0], base[0]) and torch.equal(again[1], base[1])
    plan.close()
    # layouts and dtypes without a tensor-core kernel: a rotated plan runs them on the matrix-vector kernels
    for Dv, dtv, grp, nb in [(128, "f16", 128, 4), (128, "f16", 32, 8), (160, "bf16", 32, 4)]:
        p = kb.Plan(Dv, grp, 1, bits=nb)
        Rv = wl.make_rotation(Dv, 9)
        p.set_rotation(Rv)
        xv = wl.make_vectors(5000, Dv, dtv, "gaussian", 1)
        lv = wl.make_lambda(1, Dv, 2)
        odt = ko.F16 if dtv == "f16" else ko.BF16
        pkv, scv = gpu_encode(p, xv.cuda(), lv.cuda())
        orv = ko.encode(bits(xv), odt, p.signs(), lv.numpy(), grp, want_v=True, bits=nb, rot=Rv.numpy().astype(np.float64))
        parity.check_encode(pkv.cpu().numpy(), bits(scv), orv, grp, "rotated, no tensor-core kernel", bits=nb)
        outv = gpu_decode(p, pkv, scv, lv.cuda(), dtv)
        obv, o64v = ko.decode(pkv.cpu().numpy(), bits(scv), p.signs(), lv.numpy(), grp, odt, want_f64=True, bits=nb,
                              rot=Rv.numpy().astype(np.float64))
        parity.check_decode(bits(outv), obv, o64v, odt, "rotated, no tensor-core kernel")
        p.close()


# ---- degenerate inputs: zero vectors, zero / subnormal / saturated scales, single spikes, pure tones ------------------

def _degenerate_rows(D, dtype):
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    n = torch.arange(D, dtype=torch.float64)
    rows = [torch.zeros(D, dtype=torch.float64)]                                   # scale 0, codes 0
    rows.append(torch.ones(D, dtype=torch.float64))                                # DC only
    rows.append(torch.where(n % 2 == 0, 1.0, -1.0).to(torch.float64))              # Nyquist only
    rows.append(torch.cos(2 * np.pi * 5 * n / D))                                  # one bin
    for pos, val in ((0, 1.0), (D - 1, -3.0), (D // 2, 2.0 ** -14), (7, 6.0e-8 if dtype == "f16" else 1e-30)):
        e = torch.zeros(D, dtype=torch.float64)
        e[pos] = val
        rows.append(e)                                                            # spikes: flat spectrum, down to subnormal scales
    g = torch.Generator().manual_seed(5)
    noise = torch.randn(D, generator=g, dtype=torch.float64)
    rows.append(noise * 1e-6)                                                      # fp16 scale in its subnormal range: codes are clamped
    rows.append(noise * 2e-8)                                                      # scale rounds to zero or to the smallest subnormal
    rows.append(noise * (1.5e4 if dtype == "f16" else 1e20))                       # abs-max / 7 beyond fp16: the scale saturates at 65504
    rows.append(noise * (6.0e4 / float(noise.abs().max())) if dtype == "f16" else noise * 1e30)
    rows.append(noise)
    x = torch.stack(rows).to(tdt)
    return x.repeat(23, 1)                                                         # 299 rows: three tiles, the last one ragged


@pytest.mark.parametrize("impl", ["fft", "gemm", "matvec"])
@pytest.mark.parametrize("D,dtype", [(128, "f16"), (128, "bf16"), (64, "f16"), (256, "bf16"), (160, "bf16")])
def test_degenerate_inputs(D, dtype, impl):
    odt = ko.F16 if dtype == "f16" else ko.BF16
    x = _degenerate_rows(D, dtype)
    for lam in (torch.ones(1, D), wl.make_lambda(1, D, 18), 16.0 * wl.make_lambda(1, D, 19)):   # x16: saturated scales in fp16 too
        plan = kb.Plan(D, G, 17)                                                  # a plan each: the status word is sticky
        kb.kvq_plan_set_impl(plan.handle, IMPL[impl], IMPL[impl])
        sg = plan.signs()
        packed, scales = gpu_encode(plan, x.cuda(), lam.cuda())
        assert bool(torch.isfinite(scales).all())
        ora = ko.encode(bits(x), odt, sg, lam.numpy(), G, want_v=True)
        pk, sb = packed.cpu().numpy(), bits(scales)
        # rows built to sit on the rounding grid (flat spectra, single bins, subnormal and saturated scales): the share of exact
        # ties is a property of these inputs, so the bound is 99.9 % here; every mismatch must still be off by one at a tie
        parity.check_encode(pk, sb, ora, G, "degenerate encode (%s)" % impl, min_agree=0.999)
        assert not pk[0::13].any() and not sb[0::13].any()                         # the zero vector: zero scales, zero codes
        # decode what the oracle stored, so that both sides start from the same bytes; rows whose reconstruction leaves
        # the output format's range are compared on the oracle's finite rows only
        ob, o64 = ko.decode(ora["packed"], ora["scales"], sg, lam.numpy(), G, odt, want_f64=True)
        out = gpu_decode_raw(plan, torch.from_numpy(ora["packed"]).cuda(),
                             torch.from_numpy(ora["scales"].view(np.int16)).view(torch.float16).cuda(), lam.cuda(), dtype)
        # (the tensor-core decode carries q sigma rho as an fp16 operand; rows whose scales would take it out of fp16's
        # normal range are carried times a power of two that the epilogue takes out again: they must come out right too)
        lim = 65504.0 if dtype == "f16" else 3.0e38
        ok = np.abs(o64).max(axis=1) < 0.25 * lim
        assert ok.sum() >= 0.7 * len(ok)
        # several of these rows reconstruct to values in the output format's subnormal range, where neighbouring
        # roundings are a large part of the value: the tie rule decides them, and they are not rare here by construction
        parity.check_decode(bits(out)[ok], ob[ok], o64[ok], odt, "degenerate decode (%s)" % impl, max_tie_rows=0.5)
        assert kb.kvq_plan_device_status(plan.handle) == 0
        plan.close()


@pytest.mark.parametrize("impl", ["fft", "gemm", "matvec"])
@pytest.mark.parametrize("D,dtype", [(128, "f16"), (256, "bf16"), (96, "f16")])
@pytest.mark.parametrize("wild", [False, True])
def test_degenerate_lambda(D, dtype, impl, wild):
    # mild: lambda entries spread over a factor of 100 inside a row, and a row a thousand times smaller than the other.
    # wild: entries that are zero, negative, below the 1e-6 clamp of the inverse path, or very large: the forward path
    # multiplies by them as they are, the inverse divides by max(lambda, 1e-6) (Sec. 5.1 item 1).  The tensor-core decode
    # carries 1 / lambda inside an fp16 operand next to the other channels'; a row whose reciprocals span more than 2^8
    # does not fit there, and the kernel decodes the tiles of such a row again in fp32 before it ends.  Every family is
    # held to the oracle on every row.
    odt = ko.F16 if dtype == "f16" else ko.BF16
    N = 3000
    lam = wl.make_lambda(2, D, 40)
    lam[0] = lam[0] * torch.logspace(-1, 1, D)[torch.randperm(D, generator=torch.Generator().manual_seed(1))]
    lam[1, :] = 1e-3 * lam[1, :]
    if wild:
        lam[0, 3], lam[0, 17], lam[0, 40], lam[0, D - 1], lam[0, 64] = 0.0, -1.5, 1e-8, 3e3, 1e-6
        lam[1, 5] = 2.0e-7
    x = wl.make_vectors(N, D, dtype, "k_outlier", 41)
    plan = kb.Plan(D, G, 42)
    kb.kvq_plan_set_impl(plan.handle, IMPL[impl], IMPL[impl])
    sg = plan.signs()
    packed, scales = gpu_encode(plan, x.cuda(), lam.cuda(), 1500)
    ora = ko.encode(bits(x), odt, sg, lam.numpy(), G, 1500, want_v=True)
    parity.check_encode(packed.cpu().numpy(), bits(scales), ora, G, "odd lambda encode (%s)" % impl)
    ob, o64 = ko.decode(ora["packed"], ora["scales"], sg, lam.numpy(), G, odt, 1500, want_f64=True)
    out = gpu_decode_raw(plan, torch.from_numpy(ora["packed"]).cuda(),
                         torch.from_numpy(ora["scales"].view(np.int16)).view(torch.float16).cuda(), lam.cuda(), dtype, 1500)
    assert kb.kvq_plan_device_status(plan.handle) == 0
    lim = 65504.0 if dtype == "f16" else 3.0e38
    ok = np.abs(o64).max(axis=1) < 0.25 * lim    # dividing by 1e-6 takes some rows out of fp16's range: both sides then say inf
    assert ok.sum() >= 0.3 * N
    parity.check_decode(bits(out)[ok], ob[ok], o64[ok], odt, "odd lambda decode (%s)" % impl)
    plan.close()


@pytest.mark.parametrize("D,dtype,rotated", [(128, "f16", False), (128, "bf16", False), (256, "bf16", False), (256, "f16", True), (96, "f16", False)])
def test_wide_lambda_rows_among_ordinary_ones(D, dtype, rotated):
    """The default (AUTO) decode of a call whose lambda table mixes ordinary rows with rows no fp16 operand can carry (an
    entry at the 1e-6 clamp of Sec. 5.1 item 1 next to ordinary ones, a factor 1e5 inside a row): several CTAs, segments
    that end inside a tile, a ragged last segment.  Nothing is reported and every row matches the oracle."""
    odt = DT[dtype]
    N, rpl = 20000, 3001
    n_lambda = (N + rpl - 1) // rpl
    lam = wl.make_lambda(n_lambda, D, 90)
    lam[2, 5], lam[2, D - 2] = 1e-6, 2e-7
    lam[5] = lam[5] * torch.logspace(-3, 2, D)[torch.randperm(D, generator=torch.Generator().manual_seed(2))]
    lam[n_lambda - 1, 0] = 1e-5
    plan = kb.Plan(D, G, 91)
    rot = None
    if rotated:
        R = wl.make_rotation(D, 4, 0.02)
        plan.set_rotation(R)
        rot = R.numpy().astype(np.float64)
    sg = plan.signs()
    x = wl.make_vectors(N, D, dtype, "k_outlier", 92)
    ora = ko.encode(bits(x), odt, sg, lam.numpy(), G, rpl, want_v=True, rot=rot)
    ob, o64 = ko.decode(ora["packed"], ora["scales"], sg, lam.numpy(), G, odt, rpl, want_f64=True, rot=rot)
    out = gpu_decode_raw(plan, torch.from_numpy(ora["packed"]).cuda(),
                         torch.from_numpy(ora["scales"].view(np.int16)).view(torch.float16).cuda(), lam.cuda(), dtype, rpl)
    lim = 65504.0 if dtype == "f16" else 3.0e38
    ok = np.abs(o64).max(axis=1) < 0.25 * lim
    assert ok.sum() >= 0.8 * N
    for seg in (2, 5, n_lambda - 1):                      # the wide rows keep most of their vectors inside the output range
        assert ok[seg * rpl:(seg + 1) * rpl].mean() > 0.3
    parity.check_decode(bits(out)[ok], ob[ok], o64[ok], odt, "wide lambda rows among ordinary ones")
    plan.close()


def test_rotated_d256_decode_redoes_scales_outside_its_operand_range():
    # the dense 256 x 256 kernel of rotated plans has no room for the per-row rescue: a tile with a scale its fp16 A operand
    # cannot carry is decoded again in fp32 by the same launch, so every row is held to the oracle
    D = 256
    x = _degenerate_rows(D, "bf16").repeat(8, 1)                  # 2392 rows: above the matrix-vector limit
    lam = torch.ones(1, D)
    R = wl.make_rotation(D, 3, 0.02)
    Rd = R.numpy().astype(np.float64)
    plan = kb.Plan(D, G, 17)
    plan.set_rotation(R)
    sg = plan.signs()
    packed, scales = gpu_encode(plan, x.cuda(), lam.cuda())
    ora = ko.encode(bits(x), ko.BF16, sg, lam.numpy(), G, want_v=True, rot=Rd)
    # the same grid-sitting rows as in test_degenerate_inputs: 99.9 %, every mismatch off by one at a tie
    parity.check_encode(packed.cpu().numpy(), bits(scales), ora, G, "rotated degenerate encode", min_agree=0.999)
    ob, o64 = ko.decode(ora["packed"], ora["scales"], sg, lam.numpy(), G, ko.BF16, want_f64=True, rot=Rd)
    pk_o = torch.from_numpy(ora["packed"]).cuda()
    sc_o = torch.from_numpy(ora["scales"].view(np.int16)).view(torch.float16).cuda()
    out = gpu_decode_raw(plan, pk_o, sc_o, lam.cuda(), "bf16")
    assert kb.kvq_plan_device_status(plan.handle) == 0
    sr = ko.f16_to_f64(ora["scales"])
    in_range = ((sr == 0) | ((sr >= 2.0 ** -14) & (sr <= 9357.0))).all(axis=1)
    assert 0.5 * len(in_range) <= in_range.sum() < len(in_range)        # the case does hold rows the operand cannot carry
    fin = np.abs(o64).max(axis=1) < 0.25 * 3.0e38
    parity.check_decode(bits(out)[fin], ob[fin], o64[fin], ko.BF16, "rotated degenerate decode, every row", max_tie_rows=0.5)
    parity.check_decode(bits(out)[in_range], ob[in_range], o64[in_range], ko.BF16, "rotated degenerate decode", max_tie_rows=0.5)
    plan.close()
    plan = kb.Plan(D, G, 17)
    plan.set_rotation(R)
    kb.kvq_plan_set_impl(plan.handle, kb.KVQ_IMPL_MATVEC, kb.KVQ_IMPL_MATVEC)
    out = gpu_decode_raw(plan, pk_o, sc_o, lam.cuda(), "bf16")
    assert kb.kvq_plan_device_status(plan.handle) == 0
    parity.check_decode(bits(out), ob, o64, ko.BF16, "rotated degenerate decode (matvec)", max_tie_rows=0.5)
    plan.close()


# ---- config 3: Gemma-3-1B-shaped, D = 256 bf16, prefix sweep ---------------------------------

@pytest.mark.parametrize("prefix", [256, 1024])
def test_config3_gemma_shaped_d256_bf16(prefix):
    shp = wl.GEMMA3_1B
    N = 2 * shp.layers * prefix  # K and V of every layer
    run_case(256, "bf16", N, "c1", 6000 + prefix, n_lambda=2 * shp.layers, rows_per_lambda=prefix)


def test_config3_gemma_shaped_prefix_4096_sampled():
    _full_size_sampled(256, "bf16", 2 * wl.GEMMA3_1B.layers * 4096, "c1", 6100, 2 * wl.GEMMA3_1B.layers, 4096)


# ---- beyond 2^32 bytes: row offsets must be 64-bit in every kernel family -------------------------------------------

@pytest.mark.parametrize("impl", ["gemm", "fft", "matvec"])
def test_row_offsets_beyond_four_gigabytes(impl):
    # 17,000,001 vectors of D = 128 fp16: x and x^ are 4.35 GB each, so the last rows sit past byte 2^32 of their buffers
    # (and past row 2^24); sampled rows at both ends and in between go to the oracle
    D, N = 128, 17_000_001
    n_lambda, rpl = 3, 6_000_000
    plan = kb.Plan(D, G, 23)
    kb.kvq_plan_set_impl(plan.handle, IMPL[impl], IMPL[impl])
    sg = plan.signs()
    lam = wl.make_lambda(n_lambda, D, 24)
    x = wl.make_vectors(1 << 20, D, "f16", "k_outlier", 25, device="cuda").repeat(17, 1)[:N].contiguous()   # 16 + 1 copies
    x[-4096:] = wl.make_vectors(4096, D, "f16", "gaussian", 26, device="cuda")                                # a distinct tail
    assert x.numel() * 2 > 1 << 32
    lamd = lam.cuda()
    packed, scales = gpu_encode(plan, x, lamd, rpl)
    out = gpu_decode(plan, packed, scales, lamd, "f16", rpl)
    g = torch.Generator().manual_seed(3)
    idx = torch.unique(torch.cat([torch.arange(0, 512), torch.arange(N - 1024, N), torch.randint(0, N, (2048,), generator=g),
                                  torch.arange(2 * rpl - 300, 2 * rpl + 300)]))
    idx_d = idx.cuda()
    xs, pk, sc, od = x[idx_d].cpu(), packed[idx_d].cpu().numpy(), bits(scales[idx_d]), bits(out[idx_d])
    lrow = (idx // rpl).numpy()
    mismatches = codes = 0
    for l in np.unique(lrow):
        m = lrow == l
        ora = ko.encode(bits(xs)[m], ko.F16, sg, lam.numpy()[l], G, want_v=True)
        # per lambda row: ties, scales, byte layout; the 99.99 % rule is applied to the whole sample below
        enc = parity.check_encode(pk[m], sc[m], ora, G, "rows past 4 GB, encode, lambda row %d" % l, min_agree=0.9995)
        mismatches += enc["mismatches"]
        codes += enc["codes"]
        ob, o64 = ko.decode(pk[m], sc[m], sg, lam.numpy()[l], G, ko.F16, want_f64=True)
        parity.check_decode(od[m], ob, o64, ko.F16, "rows past 4 GB, decode, lambda row %d" % l)
    assert mismatches <= (1.0 - parity.CODE_AGREEMENT) * codes, "only %.6f of the sampled codes agree" % (1.0 - mismatches / codes)
    plan.close()


# ---- config 5: Llama-3-70B-shaped: one layer's K (1,048,576 vectors) per launch, sampled rows -

def _full_size_sampled(D, dtype, N, kind, seed, n_lambda, rows_per_lambda, n_random=4096, dec_impl="auto", enc_impl="auto"):
    plan = kb.Plan(D, G, seed)
    kb.kvq_plan_set_impl(plan.handle, IMPL[enc_impl], IMPL[dec_impl])
    sg = plan.signs()
    x = wl.make_vectors(N, D, dtype, kind, seed, device="cuda")
    lam = wl.make_lambda(n_lambda, D, seed + 1, device="cuda")
    packed, scales = gpu_encode(plan, x, lam, rows_per_lambda)
    out = gpu_decode(plan, packed, scales, lam, dtype, rows_per_lambda)
    g = torch.Generator().manual_seed(seed)
    idx = torch.cat([torch.arange(0, 2048), torch.arange(N - 2048, N), torch.randint(0, N, (n_random,), generator=g)])
    idx = torch.unique(idx)
    idx_d = idx.cuda()
    lam_h = lam.cpu().numpy()
    lrow = (idx // rows_per_lambda).numpy() if n_lambda > 1 else np.zeros(len(idx), dtype=np.int64)
    xs, pk, sc, od = x[idx_d].cpu(), packed[idx_d].cpu().numpy(), bits(scales[idx_d]), bits(out[idx_d])
    mismatches = codes = 0
    tie_rows = n_rows = 0.0
    worst = 0.0
    for l in np.unique(lrow):
        m = lrow == l
        ora = ko.encode(bits(xs)[m], DT[dtype], sg, lam_h[l], G, want_v=True)
        # a lambda row's share of the sample is a few ten thousand codes: the 99.99 % rule is applied to the whole sample
        # (below), every other rule (ties, scales, byte layout) to each row's share
        enc = parity.check_encode(pk[m], sc[m], ora, G, "full-size encode lambda row %d" % l, min_agree=0.999)
        mismatches += enc["mismatches"]
        codes += enc["codes"]
        ob, o64 = ko.decode(pk[m], sc[m], sg, lam_h[l], G, DT[dtype], want_f64=True)
        dec = parity.check_decode(od[m], ob, o64, DT[dtype], "full-size decode lambda row %d" % l)
        tie_rows += dec["rows_needing_tie_rule"] * int(m.sum())
        n_rows += int(m.sum())
        worst = max(worst, dec["rel_l2_plain_max"])
    assert mismatches <= (1.0 - parity.CODE_AGREEMENT) * codes, "only %.6f of the sampled codes agree" % (1.0 - mismatches / codes)
    # how much of the decode's agreement rests on the output-rounding tie rule: little (fp16 output: none expected)
    print("full-size sampled D=%d %s dec=%s: code agreement %.6f, decode rel-L2 max %.3g, rows needing the tie rule %.4f"
          % (D, dtype, dec_impl, 1.0 - mismatches / codes, worst, tie_rows / n_rows))
    assert tie_rows / n_rows < (0.001 if dtype == "f16" else 0.02)
    # properties that hold at any size: codes in range everywhere, scales finite and non-negative
    assert bool(torch.isfinite(scales).all()) and bool((scales >= 0).all())
    lo, hi = packed & 0xF, packed >> 4
    assert not bool((lo == 8).any()) and not bool((hi == 8).any())  # -8 is never produced
    assert bool(torch.isfinite(out).all())
    plan.close()


@pytest.mark.parametrize("impl", ["fft", "gemm"])
def test_config5_llama70b_shaped_one_layer_full_size_sampled(impl):
    # the launch configuration bench.py times: K and V of one layer in one call, 2 x 1,048,576 vectors, two lambda rows
    shp = wl.LLAMA3_70B
    half = shp.kv_heads * shp.batch * shp.prefix
    _full_size_sampled(128, "f16", 2 * half, "k_outlier", 7001, 2, half, dec_impl=impl, enc_impl=impl)


def test_config5_llama70b_shaped_v_like_full_size_sampled():
    shp = wl.LLAMA3_70B
    N = shp.kv_heads * shp.batch * shp.prefix
    _full_size_sampled(128, "f16", N, "gaussian", 7002, 1, 0)
