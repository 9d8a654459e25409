"""The device quantiser computes rint(fl32(fl32(127 x) / gamma)) in IEEE binary32.  This test
replays that recipe in numpy float32 over every pair of bfloat16 mantissas and checks it against
the oracle's exact rounding (Definition "Dynamic Activation Quantization": round to nearest of
x / gamma_x * 127), so the choice of recipe is pinned without a GPU."""
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


def test_reciprocal_multiply_recipe_would_fail_on_ties():
    # documents why the kernel divides instead of multiplying by 127 / gamma
    g = np.float32(152.0)
    x = np.float32(76.0)
    exact = int(np.rint(np.float64(127.0) * np.float64(x) / np.float64(g)))   # 63.5 -> 64
    recip = int(np.rint(x * (np.float32(127.0) / g)))
    assert exact == 64 and recip == 63
