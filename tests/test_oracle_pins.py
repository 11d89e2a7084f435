"""Pins of the fp64 CPU oracle against what the paper and the mathematics fix.

None of these tests retypes the oracle's formula: each compares it with a closed
form, an invariant, a library routine (numpy rfft, numpy/torch half conversion),
brute force, or a number printed in the paper.  CPU only.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import kvq_oracle as ko
from paper_2605_05699_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
DIMS = [2, 4, 8, 12, 64, 96, 128, 160, 256]


def ones(D):
    return np.ones(D, dtype=np.int8)


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


# --------------------------------------------------------------------------
# number formats: against numpy / torch conversions (library routines)
# --------------------------------------------------------------------------

def test_f16_widen_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    got = ko.f16_to_f64(bits)
    want = bits.view(np.float16).astype(np.float64)
    both_nan = np.isnan(got) & np.isnan(want)
    assert np.array_equal(got[~both_nan], want[~both_nan])
    assert both_nan.sum() == 2 * 1023


def test_f16_narrow_matches_numpy_direct_rounding():
    r = rng(1)
    v = np.concatenate([
        r.standard_normal(20000) * np.exp(r.standard_normal(20000) * 6),
        # exact ties and neighbours around many binades, subnormal range, overflow edge
        np.array([0.0, -0.0, 2.0 ** -24, 2.0 ** -25, 1.5 * 2.0 ** -25, 2.0 ** -14, 65504.0, 65519.99, 65520.0,
                  1e6, -1e6, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 1.0 + 2.0 ** -11 + 2.0 ** -40]),
    ])
    got = ko.f64_to_f16(v)
    with np.errstate(over="ignore"):
        want = v.astype(np.float16).view(np.uint16)
    assert np.array_equal(got, want)
    # the saturating variant differs only where the plain one overflows
    sat = ko.f64_to_f16(v, saturate=True)
    over = np.abs(v) >= 65520.0
    assert np.array_equal(sat[~over], want[~over])
    assert np.all((sat[over] & 0x7FFF) == 0x7BFF)


def test_f16_narrow_every_midpoint_is_ties_to_even():
    # for each pair of adjacent positive finite halves, the exact midpoint must go to the even one
    bits = np.arange(0, 0x7BFF, dtype=np.uint16)
    lo = bits.view(np.float16).astype(np.float64)
    hi = (bits + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    mid = (lo + hi) / 2  # exact in fp64
    got = ko.f64_to_f16(mid)
    want = np.where(bits % 2 == 0, bits, bits + 1).astype(np.uint16)
    assert np.array_equal(got, want)


def test_bf16_conversions_match_torch():
    r = rng(2)
    v = r.standard_normal(20000) * np.exp(r.standard_normal(20000) * 20)
    got = ko.f64_to_bf16(v)
    want = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, want)
    back = ko.bf16_to_f64(got)
    want_back = torch.from_numpy(want.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(back, want_back)


# --------------------------------------------------------------------------
# sign diagonal: published SplitMix64 stream
# --------------------------------------------------------------------------

def _golden_stream():
    with open(os.path.join(GOLDEN, "splitmix64_seed1234567.txt")) as f:
        return [int(l) for l in f if l.strip() and not l.startswith("#")]


def test_signs_follow_published_splitmix64_stream():
    stream = _golden_stream()
    s = ko.signs(len(stream), 1234567)
    want = [-1 if (z >> 63) else 1 for z in stream]
    assert s.tolist() == want


def test_signs_are_pm1_balanced_and_seed_dependent():
    a, b = ko.signs(4096, 7), ko.signs(4096, 8)
    assert set(np.unique(a)) == {-1, 1}
    assert abs(int(a.sum())) < 4 * 64  # 4 sigma of a fair coin
    assert (a != b).mean() > 0.4
    assert np.array_equal(a[:128], ko.signs(128, 7))  # prefix property: sign n depends on (seed, n) only


# --------------------------------------------------------------------------
# transform (Eq. 1-2): invariants, closed forms, a library rfft
# --------------------------------------------------------------------------

@pytest.mark.parametrize("D", DIMS)
def test_srft_matrix_is_orthogonal(D):
    s = ko.signs(D, 11)
    M = ko.srft_forward(np.eye(D), s).T  # column n = SRFT(e_n)
    assert np.abs(M @ M.T - np.eye(D)).max() < 1e-12
    assert np.abs(M.T @ M - np.eye(D)).max() < 1e-12


@pytest.mark.parametrize("D", DIMS)
def test_srft_preserves_norms_and_inner_products_and_inverts(D):
    r = rng(D)
    s = ko.signs(D, 3)
    x, y = r.standard_normal((64, D)), r.standard_normal((64, D))
    zx, zy = ko.srft_forward(x, s), ko.srft_forward(y, s)
    assert np.abs(np.linalg.norm(zx, axis=1) / np.linalg.norm(x, axis=1) - 1).max() < 1e-12
    assert np.abs((zx * zy).sum(1) - (x * y).sum(1)).max() < 1e-11
    assert np.abs(ko.srft_inverse(zx, s) - x).max() < 1e-12
    assert np.abs(ko.srft_forward(ko.srft_inverse(x, s), s) - x).max() < 1e-12


@pytest.mark.parametrize("D", [8, 96, 128, 160, 256])
def test_srft_closed_forms_with_unit_signs(D):
    H = D // 2
    n = np.arange(D)
    s = ones(D)
    # delta at 0: flat spectrum
    z = ko.srft_forward(np.eye(D)[0], s)
    want = np.zeros(D)
    want[0] = want[H] = 1 / math.sqrt(D)
    want[1:H] = math.sqrt(2) / math.sqrt(D)
    assert np.abs(z - want).max() < 1e-14
    # constant -> DC only; alternating -> Nyquist only
    z = ko.srft_forward(np.ones(D), s)
    assert np.abs(z - math.sqrt(D) * np.eye(D)[0]).max() < 1e-12
    z = ko.srft_forward((-1.0) ** n, s)
    assert np.abs(z - math.sqrt(D) * np.eye(D)[H]).max() < 1e-12
    # pure tones: cos -> +sqrt(D/2) e_m ; sin -> -sqrt(D/2) e_{H+m}  (e^{-i...} convention)
    for m in {1, 2, H // 2, H - 1}:
        if not 1 <= m < H:
            continue
        z = ko.srft_forward(np.cos(2 * np.pi * m * n / D), s)
        assert np.abs(z - math.sqrt(D / 2) * np.eye(D)[m]).max() < 1e-12
        z = ko.srft_forward(np.sin(2 * np.pi * m * n / D), s)
        assert np.abs(z + math.sqrt(D / 2) * np.eye(D)[H + m]).max() < 1e-12


@pytest.mark.parametrize("D", DIMS)
def test_srft_equals_library_rfft_plus_eq2_repack(D):
    r = rng(100 + D)
    H = D // 2
    s = ko.signs(D, 5)
    x = r.standard_normal((32, D))
    Y = np.fft.rfft(x * s, norm="ortho", axis=1)
    want = np.empty_like(x)
    want[:, 0] = Y[:, 0].real
    want[:, H] = Y[:, H].real
    want[:, 1:H] = math.sqrt(2) * Y[:, 1:H].real
    want[:, H + 1:] = math.sqrt(2) * Y[:, 1:H].imag
    assert np.abs(ko.srft_forward(x, s) - want).max() < 1e-12
    # and the inverse against irfft
    z = r.standard_normal((32, D))
    Yz = np.zeros((32, H + 1), dtype=complex)
    Yz[:, 0] = z[:, 0]
    Yz[:, H] = z[:, H]
    Yz[:, 1:H] = (z[:, 1:H] + 1j * z[:, H + 1:]) / math.sqrt(2)
    want_x = np.fft.irfft(Yz, n=D, norm="ortho", axis=1) * s
    assert np.abs(ko.srft_inverse(z, s) - want_x).max() < 1e-12


def test_signs_act_on_the_input_side():
    # Eq. 1: F diag(s) x.  Flipping sign n must equal negating input n.
    D = 16
    r = rng(9)
    x = r.standard_normal(D)
    s = ones(D).copy()
    s[5] = -1
    x2 = x.copy()
    x2[5] = -x2[5]
    assert np.abs(ko.srft_forward(x, s) - ko.srft_forward(x2, ones(D))).max() < 1e-15


# --------------------------------------------------------------------------
# nibble layout: printed formula, brute force
# --------------------------------------------------------------------------

@pytest.mark.parametrize("n", [2, 4])
def test_nibble_pack_unpack_brute_force(n):
    vals = list(range(-8, 8))
    for q in itertools.product(vals, repeat=n):
        b = ko.pack_nibbles(np.array(q, dtype=np.int8))
        for i in range(n // 2):
            # Sec. 3.2: byte = (q[2i+1] << 4) | (q[2i] & 0xF)
            assert int(b[i]) == (((q[2 * i + 1] << 4) | (q[2 * i] & 0xF)) & 0xFF)
        assert ko.unpack_nibbles(b).tolist() == list(q)


def test_every_byte_unpacks_and_repacks():
    b = np.arange(256, dtype=np.uint8)
    q = ko.unpack_nibbles(b)
    assert q.min() == -8 and q.max() == 7
    assert np.array_equal(ko.pack_nibbles(q), b)


# --------------------------------------------------------------------------
# quantizer: scale rule, rounding rule, grid round trip, special cases
# --------------------------------------------------------------------------

def _f64_of_f16bits(b):
    return b.view(np.float16).astype(np.float64)


@pytest.mark.parametrize("D,g", [(128, 32), (256, 32), (96, 32), (160, 32), (64, 16), (128, 128)])
def test_group_maximum_maps_to_code_7_and_scale_is_absmax_over_7(D, g):
    r = rng(D + g)
    s = ko.signs(D, 1)
    lam = r.uniform(0.5, 2.0, D).astype(np.float32)
    x = r.standard_normal((200, D)) * np.exp(r.standard_normal(D))
    out = ko.encode_f64(x, s, lam, g, want_v=True)
    v = out["v"].reshape(200, D // g, g)
    q = out["codes"].reshape(200, D // g, g)
    sig = _f64_of_f16bits(out["scales"])
    a = np.abs(v).max(-1)
    # scale = absmax / (2^{b-1} - 1), stored in fp16: within half an fp16 ulp of a/7
    assert np.abs(sig / (a / 7.0) - 1).max() <= 2.0 ** -11
    # the element that attains the group maximum gets code +-7, with its sign
    idx = np.abs(v).argmax(-1)
    qmax = np.take_along_axis(q, idx[..., None], -1)[..., 0]
    vmax = np.take_along_axis(v, idx[..., None], -1)[..., 0]
    assert np.array_equal(qmax, np.where(vmax > 0, 7, -7))
    assert q.min() >= -7 and q.max() <= 7
    # v is lambda (.) SRFT(x), checked through an independent route (numpy rfft)
    H = D // 2
    Y = np.fft.rfft(x * s, norm="ortho", axis=1)
    z = np.empty_like(x)
    z[:, 0], z[:, H] = Y[:, 0].real, Y[:, H].real
    z[:, 1:H], z[:, H + 1:] = math.sqrt(2) * Y[:, 1:H].real, math.sqrt(2) * Y[:, 1:H].imag
    assert np.abs(out["v"] - z * lam.astype(np.float64)).max() < 1e-10
    # codes are the nearest grid points of the stored scale
    t = out["v"].reshape(200, D // g, g) / sig[..., None]
    assert np.abs(t - q).max() <= 0.5 + 1e-12


def test_group_equal_D_is_the_per_token_rule():
    # Sec. 3.2 step 3: one scale per vector = absmax / (2^{b-1}-1)
    D = 128
    r = rng(5)
    s = ko.signs(D, 2)
    x = r.standard_normal((50, D))
    out = ko.encode_f64(x, s, np.ones(D, np.float32), D, want_v=True)
    assert out["scales"].shape == (50, 1)
    a = np.abs(out["v"]).max(1)
    want = (a / 7.0).astype(np.float16).view(np.uint16)
    assert np.array_equal(out["scales"][:, 0], want)


def test_lambda_one_equals_unscaled_and_lambda_scales_the_rotated_vector():
    D, g = 128, 32
    r = rng(6)
    s = ko.signs(D, 4)
    x = r.standard_normal((64, D))
    lam = r.uniform(0.5, 2.0, D).astype(np.float32)
    z = ko.srft_forward(x, s)
    a = ko.encode_f64(x, s, lam, g)
    # quantizing x with lambda == quantizing the vector whose SRFT is lambda (.) z, with lambda = 1
    x_scaled = ko.srft_inverse(z * lam.astype(np.float64), s)
    b = ko.encode_f64(x_scaled, s, np.ones(D, np.float32), g)
    same = (a["codes"] == b["codes"]).mean()
    assert same > 0.9999 and np.array_equal(a["scales"], b["scales"])


@pytest.mark.parametrize("D", [96, 128, 160, 256])
def test_inputs_on_the_int4_grid_round_trip_exactly(D):
    g = 32
    r = rng(40 + D)
    s = ko.signs(D, 9)
    N = 100
    q = r.integers(-7, 8, size=(N, D)).astype(np.int8)
    # put a +-7 in every group so that the group abs-max is exactly 7 sigma
    for j in range(D // g):
        pos = r.integers(0, g, size=N) + j * g
        q[np.arange(N), pos] = r.choice([-7, 7], size=N)
    sig = np.exp(r.standard_normal((N, D // g))).astype(np.float16)
    lam = r.uniform(0.5, 2.0, D).astype(np.float32)
    packed = ko.pack_nibbles(q)
    _, x = ko.decode(packed, sig.view(np.uint16), s, lam, g, ko.F16, want_f64=True)
    out = ko.encode_f64(x, s, lam, g)
    assert np.array_equal(out["codes"], q)
    assert np.array_equal(out["scales"], sig.view(np.uint16))
    assert np.array_equal(out["packed"], packed)
    # idempotence: decode(encode(decode(.))) == decode(.)
    _, x2 = ko.decode(out["packed"], out["scales"], s, lam, g, ko.F16, want_f64=True)
    assert np.array_equal(x2, x)


def test_rounding_is_half_to_even_and_uses_the_stored_scale():
    # D = 4 with unit signs: z_0 = (x0+x1+x2+x3)/2 and z_2 = (x0-x1+x2-x3)/2 are exact in fp64
    # (their DFT rows are +-1), so exact ties can be placed there.  z_0 = 7 makes the stored scale 1.
    for tie, want in [(0.5, 0), (1.5, 2), (2.5, 2), (3.5, 4), (4.5, 4), (5.5, 6), (6.5, 6),
                      (-0.5, 0), (-1.5, -2), (-2.5, -2), (-3.5, -4), (-6.5, -6)]:
        a, b = (14 + 2 * tie) / 4, (14 - 2 * tie) / 4  # x0 = x2 = a, x1 = x3 = b
        x = np.array([[a, b, a, b]])
        out = ko.encode_f64(x, ones(4), np.ones(4, np.float32), 4, want_v=True)
        assert out["v"][0, 0] == 7.0 and out["v"][0, 2] == tie
        assert out["scales"][0, 0] == np.float16(1.0).view(np.uint16)
        assert out["codes"][0, 0] == 7 and out["codes"][0, 2] == want
    D, g = 8, 8
    s = ones(D)
    # stored (fp16-rounded) scale, not the fp64 one, decides the code:
    # a/7 = 0.1428571... rounds to fp16 0.142822265625; 6.5 sigma_fp16 is a tie only for the stored value
    z = np.zeros((1, D))
    z[0, 0] = 1.0
    sig16 = float(np.float16(1.0 / 7.0))
    z[0, 1] = 6.5 * sig16 * (1 + 1e-9)  # just above the tie of the STORED scale -> 7; for a/7 it would be 6.4996 -> 6
    x = ko.srft_inverse(z, s)
    out = ko.encode_f64(x, s, np.ones(D, np.float32), g)
    assert out["codes"][0, 1] == 7 and out["codes"][0, 0] == 7


def test_zero_group_gives_zero_scale_and_codes_and_decodes_to_zero():
    D, g = 128, 32
    s = ko.signs(D, 3)
    x = np.zeros((2, D))
    out = ko.encode_f64(x, s, np.ones(D, np.float32), g)
    assert not out["scales"].any() and not out["codes"].any() and not out["packed"].any()
    bits, x64 = ko.decode(out["packed"], out["scales"], s, np.ones(D, np.float32), g, ko.F16, want_f64=True)
    assert not x64.any() and not (bits & 0x7FFF).any()


def test_scale_saturates_at_fp16_max_and_codes_stay_in_range():
    D, g = 8, 8
    s = ones(D)
    z = np.array([[7e6, 3e6, -7e6, 1.0, 0, 0, 0, 0]])
    x = ko.srft_inverse(z, s)
    out = ko.encode_f64(x, s, np.ones(D, np.float32), g)
    assert out["scales"][0, 0] == 0x7BFF
    assert out["codes"][0].tolist()[:4] == [7, 7, -7, 0]
    # just past the last bin edge of a saturated scale: 7.8 sigma and -7.6 sigma clamp to +-7
    z = np.array([[7.8 * 65504.0, -7.6 * 65504.0, 7.4 * 65504.0, 6.6 * 65504.0, 0, 0, 0, 0]])
    out = ko.encode_f64(ko.srft_inverse(z, s), s, np.ones(D, np.float32), g)
    assert out["scales"][0, 0] == 0x7BFF
    assert out["codes"][0].tolist()[:4] == [7, -7, 7, 7]
    assert ko.unpack_nibbles(out["packed"])[0].tolist()[:4] == [7, -7, 7, 7]


def test_decode_clamps_lambda_at_1e_minus_6_and_sign_extends_minus_8():
    D, g = 8, 8
    s = ones(D)
    q = np.array([[-8, 7, 1, 0, 0, 0, 0, 0]], dtype=np.int8)
    packed = ko.pack_nibbles(q)
    sig = np.array([[1.0]], dtype=np.float16).view(np.uint16)
    lam = np.array([1.0, 1.0, 1e-9, 1, 1, 1, 1, 1], dtype=np.float32)
    _, x = ko.decode(packed, sig, s, lam, g, ko.F16, want_f64=True)
    z = ko.srft_forward(x, s)
    assert np.abs(z[0, :3] - np.array([-8.0, 7.0, 1.0 / 1e-6])).max() < 1e-6


def test_quantization_error_variance_is_lsb_squared_over_12():
    D, g = 128, 32
    r = rng(77)
    s = ko.signs(D, 5)
    x = r.standard_normal((4000, D))
    out = ko.encode_f64(x, s, np.ones(D, np.float32), g, want_v=True)
    sig = _f64_of_f16bits(out["scales"])
    err = out["v"].reshape(4000, D // g, g) - out["codes"].reshape(4000, D // g, g) * sig[..., None]
    ratio = (err ** 2).mean() / ((sig ** 2).mean() / 12)
    assert 0.9 < ratio < 1.1


def test_half_precision_entry_point_is_the_f64_path_on_widened_input():
    D, g = 128, 32
    r = rng(8)
    s = ko.signs(D, 6)
    lam = r.uniform(0.5, 2, (2, D)).astype(np.float32)
    x16 = (r.standard_normal((64, D)) * 3).astype(np.float16)
    a = ko.encode(x16, ko.F16, s, lam, g, rows_per_lambda=32)
    b0 = ko.encode_f64(x16[:32].astype(np.float64), s, lam[0], g)
    b1 = ko.encode_f64(x16[32:].astype(np.float64), s, lam[1], g)
    assert np.array_equal(a["packed"], np.concatenate([b0["packed"], b1["packed"]]))
    assert np.array_equal(a["scales"], np.concatenate([b0["scales"], b1["scales"]]))
    xb = torch.from_numpy(r.standard_normal((8, D))).to(torch.bfloat16)
    raw = xb.view(torch.int16).numpy().view(np.uint16)
    c = ko.encode(raw, ko.BF16, s, lam[0], g)
    d = ko.encode_f64(xb.to(torch.float64).numpy(), s, lam[0], g)
    assert np.array_equal(c["packed"], d["packed"])


def test_decode_output_is_the_rounded_fp64_reconstruction():
    D, g = 128, 32
    r = rng(12)
    s = ko.signs(D, 6)
    lam = r.uniform(0.5, 2, D).astype(np.float32)
    x16 = (r.standard_normal((64, D)) * 3).astype(np.float16)
    e = ko.encode(x16, ko.F16, s, lam, g)
    bits, x64 = ko.decode(e["packed"], e["scales"], s, lam, g, ko.F16, want_f64=True)
    assert np.array_equal(bits, x64.astype(np.float16).view(np.uint16))
    bb, _ = ko.decode(e["packed"], e["scales"], s, lam, g, ko.BF16, want_f64=True)
    want = torch.from_numpy(x64).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bb, want)
    # 4-bit round trip error on Gaussian data is a few percent of the norm: sanity, not a pin
    rel = np.linalg.norm(x64 - x16.astype(np.float64), axis=1) / np.linalg.norm(x16.astype(np.float64), axis=1)
    assert rel.max() < 0.25


def test_append_writes_row_pos_of_every_stream_and_nothing_else():
    D, g, S, T = 128, 32, 6, 5
    r = rng(13)
    s = ko.signs(D, 6)
    lam = r.uniform(0.5, 2, (3, D)).astype(np.float32)
    x16 = r.standard_normal((S, D)).astype(np.float16)
    pc = np.full((S, T, D // 2), 0xAB, dtype=np.uint8)
    sc = np.full((S, T, D // g), 0x1234, dtype=np.uint16)
    ko.append(x16, ko.F16, s, lam, g, pc, sc, pos=3, streams_per_lambda=2)
    e = ko.encode(x16, ko.F16, s, lam, g, rows_per_lambda=2)
    assert np.array_equal(pc[:, 3], e["packed"]) and np.array_equal(sc[:, 3], e["scales"])
    mask = np.ones(T, bool)
    mask[3] = False
    assert (pc[:, mask] == 0xAB).all() and (sc[:, mask] == 0x1234).all()


# --------------------------------------------------------------------------
# base variants: one scale per vector (g = D) and 8-bit codes (Sec. 3.2 steps 3-4, Sec. 4.1)
# --------------------------------------------------------------------------

@pytest.mark.parametrize("bits", [4, 8])
def test_two_spike_spectrum_tells_the_group_span_and_the_code_range(bits):
    # z = a e_5 + (a / 10) e_40: the spikes sit in different groups of 32.  With one scale per group both codes are
    # +-Q; with one scale per vector the small spike is rint(Q / 10): 1 for Q = 7, 13 for Q = 127.
    D, Q = 128, (1 << (bits - 1)) - 1
    s = ko.signs(D, 3)
    a = 3.0
    z = np.zeros((1, D))
    z[0, 5], z[0, 40] = a, -a / 10
    x = ko.srft_inverse(z, s)
    lam = np.ones(D, np.float32)
    e32 = ko.encode_f64(x, s, lam, 32, bits=bits)
    eD = ko.encode_f64(x, s, lam, D, bits=bits)
    assert e32["scales"].shape == (1, 4) and eD["scales"].shape == (1, 1)
    want32 = np.zeros(D, np.int8)
    want32[5], want32[40] = Q, -Q
    wantD = want32.copy()
    wantD[40] = -int(np.rint(Q / 10))
    assert np.array_equal(e32["codes"][0], want32) and np.array_equal(eD["codes"][0], wantD)
    assert eD["scales"][0, 0] == np.float16(a / Q).view(np.uint16)
    assert np.array_equal(e32["scales"][0], np.array([a / Q, a / 10 / Q, 0, 0], np.float16).view(np.uint16))
    # bytes: nibble pairs for 4 bits, the codes themselves for 8
    if bits == 8:
        assert eD["packed"].shape == (1, D) and np.array_equal(eD["packed"].view(np.int8), eD["codes"])
    else:
        assert eD["packed"].shape == (1, D // 2) and np.array_equal(ko.unpack_nibbles(eD["packed"]), eD["codes"])
    # decode: the spikes come back as code x stored scale
    _, xr = ko.decode(eD["packed"], eD["scales"], s, lam, D, ko.F16, want_f64=True, bits=bits)
    sig = float(np.float16(a / Q))
    zr = ko.srft_forward(xr, s)[0]
    want = np.zeros(D)
    want[5], want[40] = Q * sig, wantD[40] * sig
    assert np.allclose(zr, want, atol=1e-12)


@pytest.mark.parametrize("bits,g", [(4, 128), (8, 128), (8, 32)])
def test_uniform_quantizer_properties_of_the_base_variants(bits, g):
    D, N, Q = 128, 400, (1 << (bits - 1)) - 1
    r = rng(50 + bits + g)
    s = ko.signs(D, 9)
    lam = r.uniform(0.5, 2, D).astype(np.float32)
    x = r.standard_normal((N, D))
    e = ko.encode_f64(x, s, lam, g, want_v=True, bits=bits)
    v, q = e["v"], e["codes"].astype(np.float64)
    sig = ko.f16_to_f64(e["scales"]).repeat(g, axis=1)
    amax = np.abs(v).reshape(N, D // g, g).max(axis=2).repeat(g, axis=1)
    # the stored scale is absmax / Q up to its fp16 rounding; the largest coordinate of a group gets code +-Q
    assert np.all(np.abs(sig * Q - amax) <= amax * 2.0 ** -11)
    assert np.all(np.abs(q).reshape(N, D // g, g).max(axis=2) == Q) and np.abs(q).max() == Q
    # rounding to the nearest code: half a step, plus the clamp where fp16 rounded the scale down
    assert np.all(np.abs(v - q * sig) <= sig / 2 + np.maximum(amax - Q * sig, 0) + 1e-15)
    if bits == 8:   # fine steps: the error is uniform on a step, variance step^2 / 12 (textbook)
        ratio = ((v - q * sig) ** 2).mean() / (sig ** 2 / 12).mean()
        assert 0.9 < ratio < 1.1
    # the inverse undoes lambda and the transform exactly: what is lost is the rounding alone
    _, xr = ko.decode(e["packed"], e["scales"], s, lam, g, ko.F16, want_f64=True, bits=bits)
    zr = ko.srft_forward(xr, s) * lam
    assert np.allclose(zr, q * sig, atol=1e-9)


def test_a_group_of_the_whole_vector_equals_groups_of_32_that_share_their_maximum():
    # special case that reduces to the pinned g = 32 path: when every group of 32 has the same abs-max, one scale per
    # vector and one per group are the same quantizer
    D = 128
    r = rng(77)
    s = ko.signs(D, 2)
    z = r.uniform(-1, 1, (50, D))
    z[:, [3, 35, 70, 127]] = 1.5
    x = ko.srft_inverse(z, s)
    lam = np.ones(D, np.float32)
    for bits in (4, 8):
        a = ko.encode_f64(x, s, lam, 32, bits=bits)
        b = ko.encode_f64(x, s, lam, D, bits=bits)
        assert np.array_equal(a["codes"], b["codes"]) and np.array_equal(a["packed"], b["packed"])
        assert np.array_equal(a["scales"], b["scales"].repeat(4, axis=1))


# --------------------------------------------------------------------------
# learned rotation at inference (Sec. 5.1 item 2): v = lambda (.) (R z), z^ = R^T (v^ / lambda)
# --------------------------------------------------------------------------

def _random_orthogonal(D, seed):
    q, r = np.linalg.qr(rng(seed).standard_normal((D, D)))
    return q * np.sign(np.diag(r))


def test_identity_rotation_changes_nothing():
    D = 96
    s = ko.signs(D, 4)
    x = rng(60).standard_normal((40, D)).astype(np.float16)
    lam = rng(61).uniform(0.5, 2, D).astype(np.float32)
    a = ko.encode(x, ko.F16, s, lam, 32, want_v=True)
    b = ko.encode(x, ko.F16, s, lam, 32, want_v=True, rot=np.eye(D))
    assert all(np.array_equal(a[k], b[k]) for k in ("packed", "scales", "codes", "v"))
    assert np.array_equal(ko.decode(a["packed"], a["scales"], s, lam, 32, ko.F16),
                          ko.decode(a["packed"], a["scales"], s, lam, 32, ko.F16, rot=np.eye(D)))


def test_the_rotation_that_undoes_the_transform_leaves_the_plain_quantizer():
    # R = T^T for the transform matrix T (z = T x): then R z = x, and the path is the quantizer applied to lambda (.) x
    # itself; on the way out R^T = T meets the inverse transform T^T, so the output is q sigma / lambda.  A rotation
    # applied transposed, or on the wrong side of lambda, fails this.
    D = 64
    s = ko.signs(D, 12)
    R = ko.srft_forward(np.eye(D), s)          # row i = T e_i, i.e. R = T^T
    assert np.allclose(R @ R.T, np.eye(D), atol=1e-13)
    r = rng(62)
    q_true = r.integers(-7, 8, (30, D)).astype(np.float64)
    q_true[:, [0, 40]] = 7                     # every group of 32 peaks at 7: sigma = step exactly
    step = 0.25
    lam = np.where(np.arange(D) % 2 == 0, 2.0, 0.5).astype(np.float32)
    x = q_true * step / lam                    # lambda (.) x = q step, exactly (powers of two)
    e = ko.encode_f64(x, s, lam, 32, want_v=True, rot=R)
    assert np.allclose(e["v"], q_true * step, atol=1e-13)
    assert np.array_equal(e["codes"], q_true.astype(np.int8))
    assert np.all(e["scales"] == np.float16(step).view(np.uint16))
    _, xr = ko.decode(e["packed"], e["scales"], s, lam, 32, ko.F16, want_f64=True, rot=R)
    assert np.allclose(xr, x, atol=1e-13)
    # without the rotation the same input gives something else
    assert not np.array_equal(ko.encode_f64(x, s, lam, 32)["codes"], e["codes"])


def test_a_permutation_rotation_permutes_the_codes_of_a_per_vector_quantizer():
    D = 128
    s = ko.signs(D, 5)
    x = rng(63).standard_normal((25, D))
    perm = rng(64).permutation(D)
    P = np.zeros((D, D))
    P[np.arange(D), perm] = 1.0               # (P z)_i = z_perm[i]
    one = np.ones(D, np.float32)
    for nbits in (4, 8):
        a = ko.encode_f64(x, s, one, D, bits=nbits)
        b = ko.encode_f64(x, s, one, D, bits=nbits, rot=P)
        assert np.array_equal(b["codes"], a["codes"][:, perm]) and np.array_equal(a["scales"], b["scales"])


def test_an_orthogonal_rotation_keeps_norms_and_is_undone_by_its_transpose():
    D = 160
    s = ko.signs(D, 6)
    R = _random_orthogonal(D, 65)
    x = rng(66).standard_normal((20, D))
    one = np.ones(D, np.float32)
    e = ko.encode_f64(x, s, one, 32, want_v=True, rot=R)
    assert np.allclose(np.linalg.norm(e["v"], axis=1), np.linalg.norm(x, axis=1), rtol=1e-12)
    assert np.allclose(e["v"], ko.srft_forward(x, s) @ R.T, atol=1e-12)
    _, xr = ko.decode(e["packed"], e["scales"], s, one, 32, ko.F16, want_f64=True, rot=R)
    vq = e["codes"] * ko.f16_to_f64(e["scales"]).repeat(32, axis=1)
    # end to end the path is orthogonal: the reconstruction error is the rounding error, rotated
    assert np.allclose(np.linalg.norm(xr - x, axis=1), np.linalg.norm(vq - e["v"], axis=1), rtol=1e-9)
    assert np.allclose(ko.srft_forward(xr, s) @ R.T, vq, atol=1e-12)


def test_flushing_blocks_that_cover_the_prefix_equals_the_full_prefix_decode():
    # Sec. 7.2: the incremental path (flush a block, keep its dequantized rows) must leave exactly what encoding the
    # whole prefix at once and decoding all of it would give, whatever the block boundaries are
    D, g, S, T = 64, 32, 5, 23
    r = rng(41)
    s = ko.signs(D, 8)
    lam = r.uniform(0.5, 2, (3, D)).astype(np.float32)
    x16 = (r.standard_normal((S, T, D)) * 3).astype(np.float16)
    pc = np.full((S, T, D // 2), 0xCD, dtype=np.uint8)
    sc = np.full((S, T, D // g), 0x4321, dtype=np.uint16)
    dq = np.full((S, T, D), 0x7777, dtype=np.uint16)
    pos = 0
    for rows in (1, 7, 2, 8):                      # 18 of the 23 rows, ragged blocks
        ko.flush_block(x16[:, pos:pos + rows], ko.F16, s, lam, g, pc, sc, dq, pos, streams_per_lambda=2)
        pos += rows
    assert (pc[:, pos:] == 0xCD).all() and (sc[:, pos:] == 0x4321).all() and (dq[:, pos:] == 0x7777).all()
    whole = ko.encode(x16[:, :pos].reshape(-1, D), ko.F16, s, lam, g, rows_per_lambda=2 * pos)
    assert np.array_equal(pc[:, :pos].reshape(-1, D // 2), whole["packed"])
    assert np.array_equal(sc[:, :pos].reshape(-1, D // g), whole["scales"])
    full = ko.decode(whole["packed"], whole["scales"], s, lam, g, ko.F16, rows_per_lambda=2 * pos)
    assert np.array_equal(dq[:, :pos].reshape(-1, D), full)
    # a second flush over rows already written replaces them and only them
    before = dq.copy()
    ko.flush_block(x16[:, 20:22], ko.F16, s, lam, g, pc, sc, dq, 3, streams_per_lambda=2)
    changed = np.zeros(T, bool)
    changed[3:5] = True
    assert np.array_equal(dq[:, ~changed], before[:, ~changed]) and not np.array_equal(dq[:, changed], before[:, changed])
    with pytest.raises(ValueError):
        ko.flush_block(x16[:, :4], ko.F16, s, lam, g, pc, sc, dq, T - 3, streams_per_lambda=2)


# --------------------------------------------------------------------------
# numbers the paper prints about the layout
# --------------------------------------------------------------------------

def _paper_numbers():
    out = {}
    with open(os.path.join(GOLDEN, "paper_layout_numbers.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                out[k] = float(v)
    return out


def test_layout_sizes_reproduce_the_papers_compression_arithmetic():
    p = _paper_numbers()
    D, g = 128, 32
    out = ko.encode_f64(np.ones((1, D)), ones(D), np.ones(D, np.float32), g)
    packed_bytes, n_scales = out["packed"].shape[1], out["scales"].shape[1]
    assert packed_bytes == D // 2 and n_scales == D // g
    # per-token, one fp32 scale
    assert round(2 * 64 / (64 / 2 + 4), 2) == p["compression_per_token_fp32scale_d64"]
    assert round(2 * D / (packed_bytes + 4), 2) == p["compression_per_token_fp32scale_d128"]
    # g=32, fp32 scales: "int4 + 8 fp32 scales" for K and V together
    assert round(2 * (2 * D) / (2 * packed_bytes + 2 * n_scales * 4), 1) == p["compression_g32_fp32scales_d128"]
    assert 2 * n_scales == 8
    assert abs((4 * D + packed_bytes + 4) - p["bytes_per_vec_fp32in_int4_d128"]) <= 1
    assert 5 * D * math.log2(D) == p["nominal_flops_d128"]
    assert math.log2(64 / 2) == p["fft_passes_d64"] and math.log2(128 / 2) == p["fft_passes_d128"]


# ---- static lambda calibration (Sec. 7.1) -------------------------------------------------------

@pytest.mark.parametrize("D", [64, 96, 128])
def test_calibration_closed_form_on_vectors_with_known_spectra(D):
    # rows that are inverse transforms of a_c e_c have exactly one non-zero channel each: lambda_c = 1 / max a_c
    rng = np.random.default_rng(5)
    sg = ko.signs(D, 9)
    amps = rng.uniform(0.25, 4.0, size=(3, D))
    amps *= rng.choice([-1.0, 1.0], size=amps.shape)
    z = np.zeros((3 * D, D))
    for rep in range(3):
        z[rep * D + np.arange(D), np.arange(D)] = amps[rep]
    x = ko.srft_inverse(z, sg)
    # feed fp64-exact values through the fp16 entry point: keep only what fp16 holds, then compare with the same data
    xb = ko.f64_to_f16(x)
    lam, amax = ko.calibrate_lambda(xb, ko.F16, sg)
    zz = ko.srft_forward(ko.f16_to_f64(xb), sg)
    assert np.allclose(amax, np.abs(zz).max(axis=0), rtol=0, atol=0)          # the definition, on the rounded inputs
    assert np.allclose(amax, np.abs(amps).max(axis=0), rtol=2e-3)             # the construction, up to fp16 input rounding
    assert np.allclose(lam * amax, 1.0, rtol=1e-15)


def test_calibration_makes_every_channel_peak_at_one_and_is_row_order_invariant():
    D = 128
    sg = ko.signs(D, 3)
    x = wl.make_vectors(700, D, "f16", "k_outlier", 77)
    xb = wl.raw_bits(x)
    lam, amax = ko.calibrate_lambda(xb, ko.F16, sg)
    v = ko.srft_forward(ko.f16_to_f64(xb), sg) * lam
    assert np.allclose(np.abs(v).max(axis=0), 1.0, rtol=1e-14) and np.abs(v).max() <= 1.0 + 1e-14
    perm = np.random.default_rng(1).permutation(len(xb))
    lam2, _ = ko.calibrate_lambda(xb[perm], ko.F16, sg)
    assert np.array_equal(lam, lam2)
    # scaling the data by a power of two scales lambda by its inverse exactly
    lam4, _ = ko.calibrate_lambda(wl.raw_bits(x * 4), ko.F16, sg)
    assert np.array_equal(lam4 * 4, lam)
    # a channel that never carries anything gets lambda = 1
    lam0, amax0 = ko.calibrate_lambda(np.zeros((5, D), dtype=np.uint16), ko.F16, sg)
    assert np.all(lam0 == 1.0) and np.all(amax0 == 0.0)
