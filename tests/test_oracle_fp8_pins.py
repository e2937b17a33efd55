"""Pins of the oracle's FP8 (E4M3 codes + power-of-two row scale) storage functions against things
other than themselves: PyTorch's own float8_e4m3fn conversion on the CPU (another implementation
of the same published format), the format's closed forms, hand-worked rows, and properties that a
dropped case, a wrong bias, a wrong rounding direction or a wrong scale boundary would break."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_12407_b200 import inputs


def f32_to_bf16_bits(x):
    return inputs.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_code_values_match_torch_float8_and_the_closed_form():
    codes = torch.arange(256, dtype=torch.uint8)
    want = codes.view(torch.float8_e4m3fn).float().numpy()
    for c in range(256):
        if c & 0x7F == 0x7F:
            assert np.isnan(want[c])          # the two NaN codes are never produced by the encoder
            continue
        assert oracle.e4m3_value(c) == float(want[c]), c
    assert oracle.e4m3_value(0x7E) == 448.0 and oracle.e4m3_value(0xFE) == -448.0
    assert oracle.e4m3_value(0x08) == 2.0 ** -6 and oracle.e4m3_value(0x01) == 2.0 ** -9
    assert oracle.e4m3_value(0x38) == 1.0 and oracle.e4m3_value(0x3C) == 1.5


def test_encode_round_trips_every_finite_code():
    for c in range(256):
        if c & 0x7F == 0x7F:
            continue
        assert oracle.e4m3_encode(oracle.e4m3_value(c)) == c, hex(c)


def test_encode_matches_torch_on_random_and_on_ties():
    rng = np.random.default_rng(5)
    y = np.concatenate([rng.uniform(-448, 448, 4000), rng.normal(0, 1, 4000), rng.normal(0, 0.01, 2000),
                        rng.uniform(-2.0 ** -5, 2.0 ** -5, 2000)]).astype(np.float32)
    # exact midpoints between neighbouring codes: must go to the even code
    vals = np.array(sorted(oracle.e4m3_value(c) for c in range(0x7F)), dtype=np.float64)
    mids = ((vals[:-1] + vals[1:]) / 2).astype(np.float32)
    assert np.array_equal(mids.astype(np.float64), (vals[:-1] + vals[1:]) / 2)     # representable in fp32
    y = np.concatenate([y, mids, -mids])
    want = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([oracle.e4m3_encode(float(v)) for v in y], dtype=np.uint8)
    zero = (got & 0x7F) == 0          # torch and the oracle may differ in the sign of a rounded-to-zero value
    assert np.array_equal(got[~zero], want[~zero])
    assert np.all((want[zero] & 0x7F) == 0)
    for lo, hi, m in zip(vals[:-1], vals[1:], mids):
        c = oracle.e4m3_encode(float(m))
        assert c & 1 == 0 and oracle.e4m3_value(c) in (lo, hi)


def test_encode_saturates_instead_of_producing_nan_codes():
    for y in (448.0, 449.0, 463.9, 464.0, 480.0, 1e9, float("inf")):
        assert oracle.e4m3_encode(y) == 0x7E and oracle.e4m3_encode(-y) == 0xFE
    assert oracle.e4m3_encode(447.9) == 0x7E and oracle.e4m3_encode(431.9) == 0x7D   # 416 | 448, midpoint 432
    assert oracle.e4m3_encode(2.0 ** -10) == 0x00          # tie between 0 and 2^-9: to the even code 0
    assert oracle.e4m3_encode(2.0 ** -10 * 1.01) == 0x01


def row_with_amax(amax, D=128):
    x = np.zeros(D, dtype=np.float32)
    x[3] = 0.25 * amax
    x[77] = -amax
    return f32_to_bf16_bits(x)


@pytest.mark.parametrize("k", [-20, -1, 0, 3, 8, 30])
def test_scale_byte_boundaries_worked_by_hand(k):
    # amax = 1.75 * 2^k fits 448 = 1.75 * 2^8 with scale 2^(k-8); one bf16 step above needs 2^(k-7)
    codes, e = oracle.fp8_quantize_rows(row_with_amax(1.75 * 2.0 ** k)[None])
    assert int(e[0]) == k - 8 + 127 and codes[0, 77] == 0xFE and codes[0, 3] == oracle.e4m3_encode(0.25 * 448)
    codes, e = oracle.fp8_quantize_rows(row_with_amax((1.75 + 2.0 ** -7) * 2.0 ** k)[None])
    assert int(e[0]) == k - 7 + 127 and codes[0, 77] == oracle.e4m3_encode(-(1.75 + 2.0 ** -7) * 128)
    codes, e = oracle.fp8_quantize_rows(row_with_amax(1.0 * 2.0 ** k)[None])
    assert int(e[0]) == k - 8 + 127 and codes[0, 77] == oracle.e4m3_encode(-256.0)
    codes, e = oracle.fp8_quantize_rows(row_with_amax((2.0 - 2.0 ** -7) * 2.0 ** k)[None])
    assert int(e[0]) == k - 7 + 127


def test_zero_row_and_exact_values():
    codes, e = oracle.fp8_quantize_rows(np.zeros((1, 128), dtype=np.uint16))
    assert int(e[0]) == 1 and not codes.any()
    x = f32_to_bf16_bits(np.array([[448.0, -3.5, 0.015625, 0.0] * 32], dtype=np.float32))
    codes, e = oracle.fp8_quantize_rows(x)
    assert int(e[0]) == 127                                       # scale 1
    assert np.array_equal(oracle.fp8_dequantize_rows(codes, e), inputs.bf16_bits_to_f64(x))


def test_no_saturation_tight_scale_error_bound_and_projection():
    rng = np.random.default_rng(11)
    x = rng.standard_normal((500, 128)).astype(np.float32) * np.exp2(rng.integers(-12, 12, (500, 1))).astype(np.float32)
    bits = f32_to_bf16_bits(x)
    xv = inputs.bf16_bits_to_f64(bits)
    codes, e = oracle.fp8_quantize_rows(bits)
    scale = np.exp2(e.astype(np.float64) - 127)
    top = np.abs(xv).max(axis=1) / scale
    assert np.all(top <= 448.0) and np.all(top > 224.0)              # the smallest power of two that fits
    deq = oracle.fp8_dequantize_rows(codes, e)
    normal = np.abs(xv) >= scale[:, None] * 2.0 ** -6
    assert np.all(np.abs(deq - xv)[normal] <= np.abs(xv)[normal] * 2.0 ** -4)          # half a unit of 3 mantissa bits
    assert np.all(np.abs(deq - xv)[~normal] <= scale[:, None].repeat(128, 1)[~normal] * 2.0 ** -10)
    assert np.all(np.sign(deq) * np.sign(xv) >= 0)
    # stored values are bf16 numbers, and storing them again changes nothing
    stored = oracle.fp8_stored_as_bf16_bits(bits)
    assert np.array_equal(inputs.bf16_bits_to_f64(stored), deq)
    codes2, e2 = oracle.fp8_quantize_rows(stored)
    assert np.array_equal(oracle.fp8_dequantize_rows(codes2, e2), deq)
    # sign symmetry and row independence
    cneg, eneg = oracle.fp8_quantize_rows(bits ^ np.uint16(0x8000))
    assert np.array_equal(eneg, e) and np.array_equal(cneg & 0x7F, codes & 0x7F)
    c1, e1 = oracle.fp8_quantize_rows(bits[7:8])
    assert np.array_equal(c1[0], codes[7]) and e1[0] == e[7]


def test_fp8_store_appends_per_head_rows():
    rng = np.random.default_rng(3)
    k = f32_to_bf16_bits(rng.standard_normal((10, 2, 128)))
    v = f32_to_bf16_bits(rng.standard_normal((10, 2, 128)))
    st = oracle.Fp8Store(2, 128, 12)
    st.append(k[:4], v[:4]); st.append(k[4:], v[4:])
    assert st.len == 10
    for h in range(2):
        c, e = oracle.fp8_quantize_rows(np.ascontiguousarray(k[:, h]))
        assert np.array_equal(st.k[h, :10], c) and np.array_equal(st.k_scale[h, :10], e)
        c, e = oracle.fp8_quantize_rows(np.ascontiguousarray(v[:, h]))
        assert np.array_equal(st.v[h, :10], c) and np.array_equal(st.v_scale[h, :10], e)
    with pytest.raises(ValueError):
        st.append(k[:3], v[:3])
