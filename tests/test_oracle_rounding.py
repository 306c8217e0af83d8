"""Pins for the oracle's fp64 -> bf16 round-to-nearest-even helper.

The expected values come from an integer-arithmetic restatement on the fp64 bit pattern
(a different algorithm from the oracle's frexp/rint one) and from torch's fp32 -> bf16
conversion (a library routine), never from the oracle itself.
"""
import numpy as np
import torch

import oracle


def _bf16_values(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _rn_even_int(v):
    """Round float64 to bf16 by integer arithmetic on the exact rational value.

    Works for finite v whose result is a normal or subnormal bf16 (|v| < 2^128 handled,
    overflow -> inf).  Uses Python integers: exact, slow, independent.
    """
    out = np.empty(v.shape, dtype=np.uint16)
    for i, x in enumerate(v.reshape(-1)):
        x = float(x)
        sign = 0x8000 if np.signbit(x) else 0
        a = abs(x)
        if a == 0.0:
            out.reshape(-1)[i] = sign
            continue
        num, den = a.as_integer_ratio()          # exact
        # bf16 magnitudes are j * 2^-133 for j < 2^8 (subnormal/first binade) and, in binade
        # e (value in [2^e, 2^(e+1))), multiples of 2^(e-7).
        e = num.bit_length() - den.bit_length()   # first guess; fixed so that 2^e <= a < 2^(e+1)
        while (num << max(-e, 0)) < (den << max(e, 0)):
            e -= 1
        while (num << max(-(e + 1), 0)) >= (den << max(e + 1, 0)):
            e += 1
        q = max(e - 7, -133)                     # spacing exponent
        # j = a / 2^q rounded to nearest, ties to even
        n2, d2 = (num << max(-q, 0)), (den << max(q, 0))
        j, rem = divmod(n2, d2)
        if 2 * rem > d2 or (2 * rem == d2 and (j & 1)):
            j += 1
        val = j * (2.0 ** q)                      # exact: j < 2^9
        if val >= 2.0 ** 128:
            out.reshape(-1)[i] = sign | 0x7F80
            continue
        b = np.array([val], dtype=np.float32).view(np.uint32)[0] >> 16
        out.reshape(-1)[i] = sign | int(b)
    return out


def test_every_bf16_value_is_a_fixed_point():
    bits = np.arange(0, 0x7F80, dtype=np.uint16)          # all finite non-negative
    got = oracle.bf16_rn(_bf16_values(bits))
    assert np.array_equal(got, bits)
    neg = bits | 0x8000
    assert np.array_equal(oracle.bf16_rn(_bf16_values(neg)), neg)


def test_midpoints_tie_to_even_and_neighbours_round_correctly():
    bits = np.arange(0, 0x7F7F, dtype=np.uint16)
    lo, hi = _bf16_values(bits), _bf16_values(bits + 1)
    mid = (lo + hi) / 2.0                                   # exact in fp64
    got = oracle.bf16_rn(mid)
    even = np.where(bits % 2 == 0, bits, bits + 1)
    assert np.array_equal(got, even)
    below = np.nextafter(mid, -np.inf)
    above = np.nextafter(mid, np.inf)
    assert np.array_equal(oracle.bf16_rn(below), bits)
    assert np.array_equal(oracle.bf16_rn(above), bits + 1)
    # negative side mirrors
    assert np.array_equal(oracle.bf16_rn(-mid), even | 0x8000)


def test_against_integer_arithmetic_restatement():
    rng = np.random.default_rng(0)
    v = np.concatenate([
        rng.standard_normal(3000),
        rng.standard_normal(500) * 1e-39,               # bf16 subnormal range
        rng.standard_normal(500) * 1e30,
        np.array([2.0 ** -133, 2.0 ** -134, 1.5 * 2.0 ** -133, 2.0 ** -134 * 1.0000001,
                  3.3895313892515355e38, 3.4e38, 1e39, -1e39, 2.0 ** 127 * (2 - 2.0 ** -8)]),
    ])
    assert np.array_equal(oracle.bf16_rn(v), _rn_even_int(v))


def test_against_torch_on_fp32_inputs():
    # For values that are exactly fp32 there is no double rounding, so torch's fp32 -> bf16
    # conversion (round-to-nearest-even) is a valid library cross-check.
    g = torch.Generator().manual_seed(1)
    t = torch.randn(200000, generator=g, dtype=torch.float32) * torch.logspace(-20, 20, 200000)
    want = t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = oracle.bf16_rn(t.numpy().astype(np.float64))
    assert np.array_equal(got, want)


def test_single_rounding_differs_from_double_rounding():
    # 1 + 2^-8 + 2^-40 lies just above the bf16 tie at 1 + 2^-8: one rounding goes up;
    # rounding to fp32 first lands on the tie, which then goes to even (down).
    v = np.array([1.0 + 2.0 ** -8 + 2.0 ** -40])
    assert oracle.bf16_rn(v)[0] == 0x3F81
    via_fp32 = torch.tensor(v).to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)[0]
    assert via_fp32 == 0x3F80


def test_special_values():
    got = oracle.bf16_rn(np.array([0.0, -0.0, np.inf, -np.inf]))
    assert list(got) == [0x0000, 0x8000, 0x7F80, 0xFF80]
    assert (oracle.bf16_rn(np.array([np.nan]))[0] & 0x7FFF) > 0x7F80


def test_bf16_to_double_matches_c_helper():
    bits = np.arange(0, 0x7F80, dtype=np.uint32).astype(np.uint16)
    bits = np.concatenate([bits, bits | 0x8000])
    lib = oracle._load()
    py = oracle.bf16_to_double(bits)
    for i in (0, 1, 0x3F80, 0x7F7F, 0x0080, 0x7F80 + 0x3F81):
        assert lib.gmlp_oracle_bf16_to_double(int(bits[i])) == py[i]
    assert py[0x3F80] == 1.0 and py[0x7F80 + 0x4000] == -2.0 and py[1] == 2.0 ** -133
