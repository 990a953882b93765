"""Pins for the oracle's number formats: closed forms, exhaustive sweeps, and torch CPU casts."""
import numpy as np
import pytest
import torch

from oracle import sdq_oracle as so

L = so.lib()


def all_bf16_values():
    bits = np.arange(65536, dtype=np.uint16)
    vals = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).double().numpy()
    return bits, vals


def test_bf16_decode_matches_torch():
    bits, vals = all_bf16_values()
    got = np.array([L.sdqo_bf16_to_double(int(b)) for b in bits[::7]])
    ref = vals[::7]
    ok = (got == ref) | (np.isnan(got) & np.isnan(ref))
    assert ok.all()


def test_e2m1_decode_closed_form():
    for c in range(16):
        s, e, m = c >> 3, (c >> 1) & 3, c & 1
        mag = m * 0.5 if e == 0 else (1 + m / 2) * 2.0 ** (e - 1)
        v = L.sdqo_e2m1_decode(c)
        assert v == (-mag if s else mag)
        assert np.signbit(v) == bool(s)


def test_e4m3_decode_matches_torch():
    codes = torch.arange(256, dtype=torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).double().numpy()
    for c in range(256):
        if (c & 0x7F) == 0x7F:
            continue  # NaN code, never produced
        assert L.sdqo_e4m3_decode(c) == ref[c]
    assert L.sdqo_e4m3_decode(0x7E) == 448.0


def test_e8m0_decode():
    assert L.sdqo_e8m0_decode(127) == 1.0
    assert L.sdqo_e8m0_decode(0) == 2.0 ** -127
    assert L.sdqo_e8m0_decode(254) == 2.0 ** 127


def test_e2m1_encode_spot_values_ties_to_even_code():
    # midpoints go to the neighbour whose code is even
    spots = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0,
             0.2: 0.0, 0.3: 0.5, 0.7: 0.5, 1.3: 1.5, 2.4: 2.0, 2.6: 3.0, 4.9: 4.0, 5.1: 6.0,
             6.0: 6.0, 7.9: 6.0, 1e9: 6.0}
    for x, y in spots.items():
        assert L.sdqo_e2m1_decode(L.sdqo_e2m1_encode(x)) == y
        assert L.sdqo_e2m1_decode(L.sdqo_e2m1_encode(-x)) == -y
    assert L.sdqo_e2m1_encode(-0.0) == 0x8
    assert L.sdqo_e2m1_encode(-0.1) == 0x8   # sign survives rounding to zero
    assert L.sdqo_e2m1_encode(0.0) == 0x0


def e2m1_encode_thresholds(a):
    """Independent statement of E2M1 RNE: thresholds between neighbours with explicit tie directions."""
    # (midpoint, tie goes up?) between codes 0|1, 1|2, ... 6|7
    mids = [(0.25, False), (0.75, True), (1.25, False), (1.75, True), (2.5, False), (3.5, True), (5.0, False)]
    code = 0
    for i, (mid, up) in enumerate(mids):
        if a > mid or (a == mid and up):
            code = i + 1
    return code


def test_e2m1_encode_exhaustive_bf16_times_scales():
    bits, vals = all_bf16_values()
    finite = np.isfinite(vals)
    for sh in (-3, 0, 2):
        for b, v in zip(bits[finite][::3], vals[finite][::3]):
            x = float(np.ldexp(v, sh))
            want = e2m1_encode_thresholds(abs(x)) | (8 if np.signbit(x) else 0)
            assert L.sdqo_e2m1_encode(x) == want, (hex(b), x)


def test_e4m3_encode_matches_torch_cast_exhaustive():
    bits, vals = all_bf16_values()
    sel = np.isfinite(vals) & (np.abs(vals) <= 448.0)
    t = torch.from_numpy(vals[sel]).to(torch.float32)
    ref = t.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    for scale in (1.0, 0.5, 4.0):
        t2 = torch.from_numpy(vals[sel] * scale).to(torch.float32)
        ok = np.abs(vals[sel] * scale) <= 448.0
        ref = t2.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
        xs = (vals[sel] * scale)
        idx = np.nonzero(ok)[0][::2]
        got = np.array([L.sdqo_e4m3_encode(float(xs[i])) for i in idx], dtype=np.uint8)
        assert (got == ref[idx]).all()


def test_e4m3_encode_spots_and_saturation():
    assert L.sdqo_e4m3_encode(464.0) == 0x7E            # above max, saturates to 448
    assert L.sdqo_e4m3_encode(1e30) == 0x7E
    assert L.sdqo_e4m3_encode(-1e30) == 0xFE
    assert L.sdqo_e4m3_encode(-0.0) == 0x80
    assert L.sdqo_e4m3_decode(L.sdqo_e4m3_encode(2.0 ** -10)) == 0.0          # tie between 0 and 2^-9 -> even code 0
    assert L.sdqo_e4m3_decode(L.sdqo_e4m3_encode(3 * 2.0 ** -10)) == 2.0 ** -8  # tie between codes 1 and 2 -> 2
    assert L.sdqo_e4m3_decode(L.sdqo_e4m3_encode(17.0)) == 16.0  # tie 16|18 -> even mantissa (16)
    assert L.sdqo_e4m3_decode(L.sdqo_e4m3_encode(19.0)) == 20.0  # tie 18|20 -> 20


def test_encode_decode_idempotent():
    for c in range(16):
        assert L.sdqo_e2m1_encode(L.sdqo_e2m1_decode(c)) == c
    for c in range(256):
        if (c & 0x7F) == 0x7F:
            continue
        assert L.sdqo_e4m3_encode(L.sdqo_e4m3_decode(c)) == c


@pytest.mark.parametrize("j", [-20, -3, 0, 5])
def test_scale_rules_closed_forms(j):
    # amax = 6*2^j: both rules give E=j.  amax = 7*2^j: FLOOR gives j (values in (6,8) saturate), CEIL gives j+1
    assert L.sdqo_e8m0_scale_code(6.0 * 2.0 ** j, so.SCALE_OCP_FLOOR) == j + 127
    assert L.sdqo_e8m0_scale_code(6.0 * 2.0 ** j, so.SCALE_CEIL_NOSAT) == j + 127
    assert L.sdqo_e8m0_scale_code(7.0 * 2.0 ** j, so.SCALE_OCP_FLOOR) == j + 127
    assert L.sdqo_e8m0_scale_code(7.0 * 2.0 ** j, so.SCALE_CEIL_NOSAT) == j + 1 + 127
    assert L.sdqo_e8m0_scale_code(4.0 * 2.0 ** j, so.SCALE_OCP_FLOOR) == j + 127
    assert L.sdqo_e8m0_scale_code(3.99 * 2.0 ** j, so.SCALE_OCP_FLOOR) == j - 1 + 127
    assert L.sdqo_e8m0_scale_code(3.0 * 2.0 ** j, so.SCALE_CEIL_NOSAT) == j - 1 + 127
    # 8-bit operands: amax = 448*2^j -> e = j ; just above -> j+1
    assert L.sdqo_fp8_scale_exp(448.0 * 2.0 ** j) == j
    assert L.sdqo_fp8_scale_exp(449.0 * 2.0 ** j) == j + 1
    assert L.sdqo_fp8_scale_exp(224.5 * 2.0 ** j) == j


def test_scale_of_zero_block():
    assert L.sdqo_e8m0_scale_code(0.0, so.SCALE_OCP_FLOOR) == 0
    assert L.sdqo_e8m0_scale_code(0.0, so.SCALE_CEIL_NOSAT) == 0
    assert L.sdqo_fp8_scale_exp(0.0) == 0


def test_scale_exponents_clamp_to_the_e8m0_range():
    """E8M0 holds exponents -127 .. 127 (codes 0 .. 254; 255 is NaN and never produced), and the power-of-two scale of the
    8-bit operands is carried as such a code too.  Stated from that definition: whatever the rule asks for is clamped to
    the nearest representable exponent.  bf16 subnormal blocks (largest magnitude below 2^-126) reach the lower clamp."""
    # 4-bit Q-Vector scale: the floor rule wants floor(log2 a) - 2
    assert L.sdqo_e8m0_scale_code(2.0 ** -125, so.SCALE_OCP_FLOOR) == 0          # -127: the last unclamped exponent
    assert L.sdqo_e8m0_scale_code(2.0 ** -126, so.SCALE_OCP_FLOOR) == 0          # -128 -> clamped to -127
    assert L.sdqo_e8m0_scale_code(127 * 2.0 ** -133, so.SCALE_OCP_FLOOR) == 0    # the largest bf16 subnormal
    assert L.sdqo_e8m0_scale_code(2.0 ** -133, so.SCALE_OCP_FLOOR) == 0          # the smallest
    assert L.sdqo_e8m0_scale_code(2.0 ** -124, so.SCALE_OCP_FLOOR) == 1
    assert L.sdqo_e8m0_scale_code(6.0 * 2.0 ** -127, so.SCALE_CEIL_NOSAT) == 0
    assert L.sdqo_e8m0_scale_code(6.0 * 2.0 ** -140, so.SCALE_CEIL_NOSAT) == 0   # far below: still code 0
    big = float(np.float32(2.0) ** 127 * np.float32(1.9921875))                   # the largest finite bf16
    assert L.sdqo_e8m0_scale_code(big, so.SCALE_OCP_FLOOR) == 125 + 127          # floor(log2) - 2 = 125: inside the range
    assert L.sdqo_e8m0_scale_code(big, so.SCALE_CEIL_NOSAT) == 126 + 127         # 6 * 2^126 >= big > 6 * 2^125
    # 8-bit operands: smallest e with a <= 448 * 2^e
    assert L.sdqo_fp8_scale_exp(448.0 * 2.0 ** -127) == -127                     # exactly representable at the bound
    assert L.sdqo_fp8_scale_exp(447.0 * 2.0 ** -127) == -127
    assert L.sdqo_fp8_scale_exp(448.0 * 2.0 ** -128) == -127                     # would be -128: clamped
    assert L.sdqo_fp8_scale_exp(2.0 ** -133) == -127
    assert L.sdqo_fp8_scale_exp(big) == 120                                      # 448 * 2^119 = 1.75 * 2^127 < big <= 448 * 2^120
    assert L.sdqo_fp8_scale_exp(1e300) == 127                                    # beyond every bf16: the upper clamp
