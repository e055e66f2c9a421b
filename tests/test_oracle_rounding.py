"""Pins for the oracle's bf16 storage rounding (CPU only): hand-computed cases of round to nearest,
ties to even, and agreement with torch's own float32 -> bfloat16 conversion."""
import numpy as np

from oracle.rounding import round_to_bf16
import seeded_inputs as si


def test_hand_computed_cases():
    e = 2.0 ** -8                      # half of bf16's spacing just above 1.0 (spacing 2^-7)
    cases = {
        1.0: 1.0,
        1.0 + e: 1.0,                  # tie -> even mantissa (1.0)
        1.0 + 3 * e: 1.0 + 4 * e,      # tie -> even mantissa (1 + 2^-6)
        1.0 + e * 1.01: 1.0 + 2 * e,   # above the tie
        1.0 + e * 0.99: 1.0,           # below the tie
        -2.5: -2.5,
        0.0: 0.0,
    }
    for x, want in cases.items():
        got = float(round_to_bf16(np.array([x]))[0])
        assert got == want, (x, got, want)
    # 8 significant bits: every result has at most 8 significant bits
    z = si.normal_f64(3, "r", 1000)
    r = round_to_bf16(z)
    m, _ = np.frexp(r)
    assert np.all(m * 256 == np.round(m * 256))
    assert np.max(np.abs(r - z) / np.abs(z)) <= 2.0 ** -8 * (1 + 1e-6)


def test_agrees_with_torch_conversion():
    import torch
    z = si.normal_f64(4, "t", 20000) * np.exp(si.normal_f64(5, "s", 20000) * 5)
    want = torch.from_numpy(z.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(round_to_bf16(z), want)
    # and with the input generator's rounding (independent implementation)
    assert np.array_equal(si.bf16_bits_to_f64(si.round_to_bf16_bits(z)), want)
