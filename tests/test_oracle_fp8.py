"""Pins for the FP8 E4M3 codec of the oracle: torch's float8_e4m3fn conversions (a library routine),
the format's closed-form landmarks, and order / round-trip properties."""
import numpy as np
import torch

from oracle import fp8


def torch_decode(codes):
    return torch.from_numpy(np.asarray(codes, dtype=np.uint8)).view(torch.float8_e4m3fn).to(torch.float64).numpy()


def torch_encode(x):
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()


def test_decode_all_codes_against_library():
    codes = np.arange(256, dtype=np.uint8)
    mine, ref = fp8.decode(codes), torch_decode(codes)
    np.testing.assert_array_equal(np.isnan(mine), np.isnan(ref))
    ok = ~np.isnan(ref)
    np.testing.assert_array_equal(mine[ok], ref[ok])


def test_format_landmarks():
    assert fp8.decode([0x7e])[0] == 448.0                 # largest finite: 1.75 * 2^8
    assert fp8.decode([0x01])[0] == 2.0 ** -9             # smallest subnormal
    assert fp8.decode([0x08])[0] == 2.0 ** -6             # smallest normal
    assert fp8.decode([0x38])[0] == 1.0
    assert fp8.decode([0xb8])[0] == -1.0
    assert np.isnan(fp8.decode([0x7f])[0]) and np.isnan(fp8.decode([0xff])[0])
    assert fp8.decode([0x00])[0] == 0.0


def test_round_trip_of_every_finite_code():
    codes = np.array([c for c in range(256) if c & 0x7f != 0x7f], dtype=np.uint8)
    again = fp8.encode(fp8.decode(codes))
    keep = codes != 0x80                                   # -0 decodes to -0.0 and comes back with its sign
    np.testing.assert_array_equal(again[keep], codes[keep])
    assert again[codes == 0x80][0] in (0x00, 0x80)


def test_encode_against_library_random_and_ties():
    rng = np.random.default_rng(8)
    x = np.concatenate([rng.normal(size=20000) * s for s in (1e-3, 0.05, 1.0, 30.0, 400.0)]).astype(np.float32)
    x = x[np.abs(x) < 464.0]           # the library does not saturate (it gives NaN beyond the range); see below
    np.testing.assert_array_equal(fp8.encode(x.astype(np.float64)), torch_encode(x))
    # exact midpoints between neighbours (ties go to the even mantissa), both signs
    vals = np.sort(fp8.decode(np.array([c for c in range(0x7f)], dtype=np.uint8)))
    mids = ((vals[:-1] + vals[1:]) / 2).astype(np.float32)
    both = np.concatenate([mids, -mids])
    np.testing.assert_array_equal(fp8.encode(both.astype(np.float64)), torch_encode(both))


def test_saturation_and_order():
    big = np.array([449.0, 1e6, -1e6, 464.0, 480.0], dtype=np.float64)
    np.testing.assert_array_equal(fp8.decode(fp8.encode(big)), [448.0, 448.0, -448.0, 448.0, 448.0])
    x = np.linspace(-500, 500, 4001)
    d = fp8.decode(fp8.encode(x))
    assert (np.diff(d) >= 0).all()                         # monotone
    inside = np.abs(x) <= 448
    assert (np.abs(d[inside] - x[inside]) <= np.maximum(np.abs(x[inside]) / 16, 2.0 ** -10)).all()   # half a step


def test_quantise_rows_uses_a_float32_product():
    rows = np.array([0.1, -2.5, 3.14159, 100.0])
    scale, inv = np.float32(0.37), np.float32(1.0) / np.float32(0.37)
    codes, deq = fp8.quantise_rows(rows, scale, inv)
    want = torch_encode(rows.astype(np.float32) * inv)
    np.testing.assert_array_equal(codes, want)
    np.testing.assert_array_equal(deq, torch_decode(want) * float(scale))
