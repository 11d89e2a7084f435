"""Parity rules between the CUDA path and the fp64 oracle, written once.

Tolerances (the project's stated ones, with the readings the design notes list):
  * nibble pack / unpack: bit-exact (GPU bytes unpack to the GPU's own codes and repack to the same bytes;
    where codes agree the bytes agree).
  * int4 codes: identical on >= 99.99 % of the entries of a tensor (a caller that splits one tensor into small
    subsamples passes a looser per-subsample bound and applies 99.99 % to the whole); every mismatch is off by exactly one and lies at a
    rounding tie: with t = v_oracle / sigma in fp64, |t - boundary| <= 1e-3 for sigma = the GPU's or the
    oracle's stored scale; or, when the two stored scales differ (by one fp16 ulp at most), the GPU code is
    the correctly rounded code for the GPU's own stored scale.
  * group scales: |sigma_gpu - sigma_oracle| <= 1 fp16 ulp everywhere, and relative L2 per vector <= 1e-3.
  * reconstruction: relative L2 per vector <= 1e-3 against the oracle's output rounded to the same dtype,
    not counting elements where the two outputs are format neighbours and the exact value sits at the
    midpoint between them (within 1e-3 of the vector's rms): the output format's own rounding tie.
"""
from __future__ import annotations

import numpy as np

from oracle import kvq_oracle as ko

CODE_AGREEMENT = 0.9999
TIE_TOL = 1e-3
REL_L2 = 1e-3


def f16_bits_to_f64(b):
    return np.ascontiguousarray(b).view(np.uint16).view(np.float16).astype(np.float64)


def check_encode(gpu_packed, gpu_scales_bits, ora, group, label="", bits=4, min_agree=CODE_AGREEMENT):
    """gpu_packed [N, D bits/8] uint8, gpu_scales_bits [N,G] uint16, ora = oracle.encode(..., want_v=True, bits=bits).
    The rules are those of the 4-bit codes with 7 read as 2^(bits-1) - 1; 8-bit codes are one byte each."""
    gpu_packed = np.ascontiguousarray(gpu_packed).view(np.uint8)
    gpu_scales_bits = np.ascontiguousarray(gpu_scales_bits).view(np.uint16)
    Q = (1 << (bits - 1)) - 1
    N = gpu_packed.shape[0]
    D = gpu_packed.shape[1] * 8 // bits
    G = D // group
    q_or = ora["codes"]
    if bits == 4:
        q_gpu = ko.unpack_nibbles(gpu_packed)
        # pack/unpack bit-exactness
        assert np.array_equal(ko.pack_nibbles(q_gpu), gpu_packed), label + ": repacking the GPU codes changes bytes"
    else:
        q_gpu = gpu_packed.view(np.int8)
    assert q_gpu.min(initial=0) >= -Q and q_gpu.max(initial=0) <= Q, label + ": code outside [-%d, %d]" % (Q, Q)
    same = q_gpu == q_or
    byte_same = gpu_packed == ora["packed"]
    if bits == 4:
        assert np.array_equal(byte_same, same[:, 0::2] & same[:, 1::2]), label + ": byte layout disagrees with codes"
    else:
        assert np.array_equal(byte_same, same), label + ": byte layout disagrees with codes"

    # scales
    bg = gpu_scales_bits.astype(np.int64)
    bo = ora["scales"].astype(np.int64)
    assert np.abs(bg - bo).max(initial=0) <= 1, label + ": a scale differs by more than one fp16 ulp"
    sg, so = f16_bits_to_f64(gpu_scales_bits), f16_bits_to_f64(ora["scales"])
    den = np.linalg.norm(so, axis=1)
    rel = np.linalg.norm(sg - so, axis=1) / np.where(den > 0, den, 1.0)
    assert rel.max(initial=0) <= REL_L2, label + ": scales relative L2 %.3g" % rel.max()
    scale_flip_frac = float((bg != bo).mean()) if bg.size else 0.0
    assert scale_flip_frac < 0.01, label + ": %.3g of the scales differ" % scale_flip_frac

    # codes
    agree = float(same.mean()) if same.size else 1.0
    assert agree >= min_agree, label + ": only %.6f of the codes agree" % agree
    rr, cc = np.nonzero(~same)
    if rr.size:
        v = ora["v"][rr, cc]
        qg = q_gpu[rr, cc].astype(np.int64)
        qo = q_or[rr, cc].astype(np.int64)
        assert np.all(np.abs(qg - qo) == 1), label + ": a code differs by more than one"
        boundary = (qg + qo) / 2.0
        s_g, s_o = sg[rr, cc // group], so[rr, cc // group]
        with np.errstate(divide="ignore", invalid="ignore"):
            t_g, t_o = v / s_g, v / s_o
        at_tie = (np.abs(t_g - boundary) <= TIE_TOL) | (np.abs(t_o - boundary) <= TIE_TOL)
        own = (s_g != s_o) & (np.clip(np.rint(t_g), -Q, Q) == qg)
        bad = ~(at_tie | own)
        assert not bad.any(), label + ": %d mismatched codes are not at a rounding tie (e.g. t=%r)" % (
            bad.sum(), t_o[bad][:4])
    return {"agree": agree, "mismatches": int(rr.size), "codes": int(same.size), "scale_flips": scale_flip_frac,
            "scale_rel_l2": float(rel.max(initial=0))}


def rel_l2_rows(a, b):
    den = np.linalg.norm(b, axis=1)
    num = np.linalg.norm(a - b, axis=1)
    return np.where(den > 0, num / np.where(den > 0, den, 1.0), num)


def check_decode(gpu_bits, ora_bits, ora_f64, dtype, label="", max_tie_rows=0.05):
    """gpu_bits / ora_bits: raw uint16 bits of the half-precision outputs [N, D]; ora_f64: the oracle's
    reconstruction before its rounding to the output dtype.

    A vector passes if its relative L2 distance to the oracle's rounded output is <= 1e-3.  The 16-bit
    output format decides a rounding, like the quantizer decides a code: two correct results can differ
    by one output ulp on an element whose exact value sits at a rounding midpoint, and for bfloat16 one
    such flip on a dominant channel is already 4e-3 of the vector norm.  A vector that fails the plain
    comparison is therefore compared again without the elements where the two outputs are neighbours in
    the format and the exact value lies within 1e-3 of the vector's rms from their midpoint; it must
    then pass, and such vectors must be rare (``max_tie_rows``; a test made of vectors whose outputs sit in the format's
    subnormal range, where one ulp is a large part of the value, raises it).
    """
    gb = np.ascontiguousarray(gpu_bits).view(np.uint16)
    g = ko.widen(gb, dtype)
    o = ko.widen(ora_bits, dtype)
    assert np.isfinite(g).all(), label + ": non-finite output"
    D = g.shape[1]
    plain = rel_l2_rows(g, o)
    need = plain > REL_L2
    worst = float(plain[~need].max(initial=0))
    if need.any():
        gg, oo, x64 = g[need], o[need], ora_f64[need]
        rms = np.linalg.norm(x64, axis=1, keepdims=True) / np.sqrt(D)
        # neighbours in the format: sign-magnitude bit patterns one apart (or +-0)
        key = lambda b: np.where(b & 0x8000, -(b & 0x7FFF).astype(np.int64), (b & 0x7FFF).astype(np.int64))
        adjacent = np.abs(key(gb[need]) - key(ora_bits[need])) == 1
        at_tie = adjacent & (np.abs(x64 - (gg + oo) / 2) <= REL_L2 * rms)
        diff = np.where(at_tie, 0.0, gg - oo)
        den = np.linalg.norm(oo, axis=1)
        rel = np.linalg.norm(diff, axis=1) / np.where(den > 0, den, 1.0)
        assert rel.max() <= REL_L2, label + ": reconstruction relative L2 %.3g (plain %.3g)" % (rel.max(), plain.max())
        worst = max(worst, float(rel.max()))
    frac = float(need.mean()) if need.size else 0.0
    assert frac < max_tie_rows, label + ": %.3g of the vectors pass only with the output-tie rule" % frac
    return {"rel_l2_max": worst, "rel_l2_plain_max": float(plain.max(initial=0)),
            "rel_l2_plain_mean": float(plain.mean()) if plain.size else 0.0, "rows_needing_tie_rule": frac,
            "bit_equal": float((gb == ora_bits).mean()) if g.size else 1.0}
