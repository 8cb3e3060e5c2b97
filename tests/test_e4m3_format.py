"""The E4M3 inputs of the FP8 paths reach the oracle through torch's float8_e4m3fn widening.
This pins that widening to the format's definition (OCP 8-bit floating point, E4M3: 1 sign bit,
4 exponent bits with bias 7, 3 mantissa bits, subnormals, no infinities, NaN = S.1111.111),
code by code, so the oracle's inputs do not rest on the library alone."""
import math

import torch


def decode_e4m3(code: int) -> float:
    sign = -1.0 if code & 0x80 else 1.0
    e = (code >> 3) & 0xF
    m = code & 0x7
    if e == 0xF and m == 0x7:
        return math.nan
    if e == 0:
        return sign * (m / 8.0) * 2.0 ** -6          # subnormal
    return sign * (1.0 + m / 8.0) * 2.0 ** (e - 7)


def test_all_256_codes():
    codes = torch.arange(256, dtype=torch.uint8)
    got = codes.view(torch.float8_e4m3fn).double()
    n_nan = 0
    for c in range(256):
        want = decode_e4m3(c)
        if math.isnan(want):
            assert math.isnan(got[c].item()), c
            n_nan += 1
        else:
            assert got[c].item() == want, (c, got[c].item(), want)
    assert n_nan == 2
    assert got[0x7e].item() == 448.0 and got[0x01].item() == 2.0 ** -9      # largest finite, smallest subnormal


def test_rounding_to_e4m3_is_nearest_even():
    """The input recipe rounds fp32 draws to E4M3 with torch: ties go to the even code, values
    beyond 448 do not become infinite."""
    x = torch.tensor([1.0625, 1.1875, 0.0009765625, 0.0029296875, 17.0, 19.0, 464.0], dtype=torch.float32)
    got = x.to(torch.float8_e4m3fn).double().tolist()
    # 1.0625 is midway between 1.0 and 1.125 -> 1.0 (even mantissa); 1.1875 midway 1.125 / 1.25 -> 1.25
    assert got[0] == 1.0 and got[1] == 1.25
    # 2^-10 is midway between 0 and the smallest subnormal 2^-9 -> 0 (even); 3 * 2^-10 -> 2^-8
    assert got[2] == 0.0 and got[3] == 2.0 ** -8
    # 17 midway between 16 and 18 -> 16; 19 midway between 18 and 20 -> 20
    assert got[4] == 16.0 and got[5] == 20.0
    assert math.isfinite(got[6]) or math.isnan(got[6])
