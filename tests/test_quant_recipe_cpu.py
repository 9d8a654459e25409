"""Pins, without a GPU, the two rounding recipes of the device quantiser against the oracle's exact
rounding (Definition "Dynamic Activation Quantization": round to nearest, ties to even, of
x / gamma_x * 127), over every pair of bfloat16 significands and every exponent gap that can
yield a nonzero code.

1. The division recipe, rint(fl32(fl32(127 x) / gamma)) in IEEE binary32: what the kernels use
   when the scale is the 1e-5 floor (the only scale that is not itself a bfloat16 value).
2. The division-free recipe every other row takes: candidate q from one fma with the constant
   1.5 * 2^23 (the sum's low mantissa bits hold q), the residual 127 x - q gamma from a second fma,
   and a tie (2 |residual| = gamma with q odd) moved one step towards the residual's sign.  It is
   replayed here in exact rational arithmetic, each fma rounded once to binary32, and the
   statements the kernel relies on are checked on the way: the residual is exactly representable,
   2 |residual| never exceeds gamma, and the code's low byte is the low byte of the sum's bit pattern.
"""
from fractions import Fraction

import numpy as np

import oracle
from paper_2602_05269_b200 import inputs as syn


def test_fp32_division_recipe_is_exact_for_all_bf16_mantissa_pairs():
    # x = mx * 2^ex, gamma = mg * 2^eg with 8-bit significands 128..255; x <= gamma.
    mant = np.arange(128, 256, dtype=np.float32)
    mismatches = 0
    total = 0
    for ex in range(-9, 1):                      # x / gamma from 2^-9 up to 1
        xs = mant * np.float32(2.0 ** ex)
        for g in mant:
            row = np.zeros((1, 192), np.float32)
            row[0, 0] = g
            row[0, 1:129] = xs
            row[0, 129:] = 0
            keep = row[0] <= g
            row[0, ~keep] = 0
            bits = syn.f32_to_bf16_bits(row)
            assert np.array_equal(syn.bf16_bits_to_f32(bits), row)
            xq, gx = oracle.act_quant(bits)
            recipe = np.rint((np.float32(127.0) * row) / np.float32(g)).astype(np.int32)
            recipe = np.clip(recipe, -127, 127)
            mismatches += int((recipe[0] != xq[0]).sum())
            total += 192
    assert total > 200000 and mismatches == 0


def _fl32(v: Fraction) -> Fraction:
    """Round a rational to the nearest binary32 value (ties to even); normal range only."""
    if v == 0:
        return v
    sign, a = (-1 if v < 0 else 1), abs(v)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    ulp = Fraction(2) ** (e - 23)
    return sign * round(a / ulp) * ulp          # round(Fraction) rounds half to even


def test_division_free_recipe_in_exact_arithmetic_matches_the_oracle():
    magic = Fraction(12582912)                   # 1.5 * 2^23
    ties = moved = total = 0
    for mg in range(128, 256):                   # gamma = mg (the recipe is invariant under powers of two)
        gamma = Fraction(mg)
        inv127 = _fl32(Fraction(127) / gamma)    # __fdiv_rn(127, gamma)
        row = [mg] + [mx * 2.0 ** ex for ex in range(-11, 1) for mx in range(128, 256) if mx * 2.0 ** ex <= mg]
        row += [-v for v in row[1:200]]
        pad = (-len(row)) % 64
        arr = np.array(row + [0.0] * pad, np.float32)[None, :]
        bits = syn.f32_to_bf16_bits(arr)
        assert np.array_equal(syn.bf16_bits_to_f32(bits), arr)
        want, gx = oracle.act_quant(bits)
        assert gx[0] == np.float32(mg)
        for i, xv in enumerate(row):
            x = Fraction(xv)
            tm = _fl32(x * inv127 + magic)                       # fmaf(x, inv127, magic)
            q = tm - magic                                       # magic - tm is exact in binary32
            assert q.denominator == 1 and abs(q) <= 127
            res_exact = 127 * x - q * gamma
            res = _fl32(res_exact)                               # fmaf(magic - tm, gamma, 127 x)
            assert res == res_exact                              # ... which is exact
            assert 2 * abs(res) <= gamma                         # the candidate is at most a tie away
            # the kernel takes the code's byte from the bit pattern of tm: mantissa = 2^22 + q
            pattern = (int(tm) - (1 << 23)) | (150 << 23)
            assert (pattern & 0xFF) == (int(q) & 0xFF)
            code = int(q)
            if 2 * abs(res) == gamma:
                ties += 1
                if code & 1:
                    code += 1 if res > 0 else -1
                    moved += 1
            assert code == int(want[0, i]), (mg, xv, code, int(want[0, i]))
            total += 1
    assert total > 150000 and ties > 0 and moved > 0


def test_reciprocal_multiply_recipe_would_fail_on_ties():
    # why neither recipe is a bare multiplication by 127 / gamma
    g = np.float32(152.0)
    x = np.float32(76.0)
    exact = int(np.rint(np.float64(127.0) * np.float64(x) / np.float64(g)))   # 63.5 -> 64
    recip = int(np.rint(x * (np.float32(127.0) / g)))
    assert exact == 64 and recip == 63
