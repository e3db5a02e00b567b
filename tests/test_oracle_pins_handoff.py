"""Pins for the compressed hand-off codec of the oracle (8-bit codes, one scale per token).

The format is fixed by its definition (4 exponent bits with bias 7, 3 mantissa bits, subnormals, no
infinities, largest finite value 448); the pins are the values that definition prints, properties
that hold for any correct nearest-even encoder, and torch's own CPU conversion to the same format
as an independent routine.
"""
import numpy as np
import torch

from oracle import handoff_codec as Q


def test_format_defining_values():
    t = Q.e4m3_table()
    assert t[0x00] == 0.0 and t[0x80] == 0.0 and np.signbit(t[0x80])
    assert t[0x01] == 2.0 ** -9            # smallest subnormal
    assert t[0x07] == 7 * 2.0 ** -9        # largest subnormal
    assert t[0x08] == 2.0 ** -6            # smallest normal
    assert t[0x38] == 1.0
    assert t[0x40] == 2.0
    assert t[0x7E] == 448.0                # largest finite
    assert np.isnan(t[0x7F]) and np.isnan(t[0xFF])
    assert np.all(np.diff(t[:0x7F]) > 0)   # codes 0x00..0x7E increase strictly
    assert np.array_equal(t[0x80:0xFF], -t[0x00:0x7F])


def test_round_trip_over_all_finite_codes():
    codes = np.array([c for c in range(256) if c & 0x7F != 0x7F], dtype=np.uint8)
    vals = Q.e4m3_table()[codes].astype(np.float32)
    assert np.array_equal(Q.e4m3_encode(vals), codes)


def test_halfway_cases_go_to_the_even_code_and_neighbours_to_the_nearer():
    t = Q.e4m3_table()
    for c in range(0x00, 0x7E):
        mid = np.float32((t[c] + t[c + 1]) / 2)          # exact in fp32
        assert (t[c] + t[c + 1]) / 2 == float(mid)
        want = c if c % 2 == 0 else c + 1
        assert Q.e4m3_encode([mid])[0] == want, hex(c)
        below, above = np.nextafter(mid, np.float32(0)), np.nextafter(mid, np.float32(1e9))
        assert Q.e4m3_encode([below])[0] == c and Q.e4m3_encode([above])[0] == c + 1
        assert Q.e4m3_encode([-mid])[0] == (want | 0x80)


def test_saturation_and_monotonicity():
    assert list(Q.e4m3_encode(np.float32([448.0, 449.0, 1e6, -1e6, 463.9]))) == [0x7E, 0x7E, 0x7E, 0xFE, 0x7E]
    y = np.sort(np.random.default_rng(0).uniform(-460, 460, 20000).astype(np.float32))
    v = Q.e4m3_table()[Q.e4m3_encode(y)]
    assert np.all(np.diff(v) >= 0)


def test_against_torch_cpu_conversion():
    rng = np.random.default_rng(1)
    y = np.concatenate([rng.uniform(-448, 448, 50000), rng.normal(0, 1, 50000), rng.normal(0, 0.01, 50000),
                        rng.uniform(-2 ** -6, 2 ** -6, 20000)]).astype(np.float32)
    y = y[np.abs(y) <= 448]
    ref = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(Q.e4m3_encode(y), ref)
    back = torch.from_numpy(ref).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    assert np.array_equal(Q.e4m3_table()[ref].astype(np.float32), back)


def test_row_scaling_error_bound_and_exact_maximum():
    rng = np.random.default_rng(2)
    x = (rng.normal(0, 1, (64, 768)) * rng.uniform(1e-6, 30, (64, 1))).astype(np.float32)
    x[5] = 0.0
    codes, scales = Q.quantize_rows(x)
    xh = Q.dequantize_rows(codes, scales, bf16=False)
    absmax = np.abs(x).max(axis=1)
    assert scales[5] == 0 and np.all(codes[5] == 0) and np.all(xh[5] == 0)
    # the largest element of a row maps to +-448 and comes back within fp32 rounding
    j = np.abs(x).argmax(axis=1)
    rows = np.arange(64)
    assert np.all((codes[rows, j] & 0x7F)[absmax > 0] == 0x7E)
    assert np.allclose(xh[rows, j], x[rows, j], rtol=3e-7, atol=0)
    # nearest-value rounding: half a step of the format, relative 2^-4 for normals, absolute
    # 2^-10 (in units of the scale) below the smallest normal
    bound = np.maximum(np.abs(x) * 2.0 ** -4, absmax[:, None] / 448 * 2.0 ** -10) * (1 + 1e-5)
    assert np.all(np.abs(xh - x) <= bound)
    # scale invariance: a power-of-two multiple of a row has the same codes
    c2, s2 = Q.quantize_rows(x * np.float32(8))
    assert np.array_equal(c2, codes) and np.array_equal(s2, scales * 8)


def test_bf16_rounding_of_the_restored_values():
    v = np.float32([1.0, 1.00390625, 1.01171875, -3.14159, 1e-30])    # 1 + 2^-8 is a tie -> 1.0; 1 + 3*2^-8 -> 1 + 2^-6
    ref = torch.from_numpy(v).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(Q.round_to_bf16(v), ref)
    y = np.random.default_rng(3).normal(0, 5, 10000).astype(np.float32)
    assert np.array_equal(Q.round_to_bf16(y), torch.from_numpy(y).to(torch.bfloat16).to(torch.float32).numpy())
