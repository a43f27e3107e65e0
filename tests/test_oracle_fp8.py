"""Pins for the FP8 cache's number format as the oracle decodes it: hand values of the e4m3 encoding, a
library decoder (torch.float8_e4m3fn), monotonicity, and the single rounding of the dequantised value."""
import numpy as np
import torch

import oracle
from paper_2608_30252_b200 import inputs


def test_e4m3_hand_values():
    bits = np.array([0x00, 0x01, 0x07, 0x08, 0x38, 0x3C, 0x40, 0x7E, 0x80, 0xC0, 0xFE], dtype=np.uint8)
    want = [0.0, 2.0 ** -9, 7 * 2.0 ** -9, 2.0 ** -6, 1.0, 1.5, 2.0, 448.0, -0.0, -2.0, -448.0]
    got = oracle.e4m3_to_f64(bits)
    assert np.array_equal(got, np.array(want))
    assert np.isnan(oracle.e4m3_to_f64(np.array([0x7F, 0xFF], dtype=np.uint8))).all()


def test_e4m3_decode_equals_the_library_decoder_on_all_256_bytes():
    bits = np.arange(256, dtype=np.uint8)
    lib = torch.from_numpy(bits).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = oracle.e4m3_to_f64(bits)
    assert np.array_equal(np.isnan(got), np.isnan(lib))
    assert np.array_equal(got[~np.isnan(got)], lib[~np.isnan(lib)])
    pos = got[:0x7F]
    assert (np.diff(pos) > 0).all()                              # the positive codes are strictly increasing


def test_dequantised_value_is_one_fp16_rounding_of_the_exact_product():
    rng = np.random.default_rng(5)
    bits = rng.integers(0, 256, 4096).astype(np.uint8)
    bits = bits[(bits & 0x7F) != 0x7F]
    scale = np.float32(0.0123)
    got = oracle.dequantize_e4m3(bits, scale)
    exact = oracle.e4m3_to_f64(bits) * float(np.float16(scale))
    assert np.array_equal(got, exact.astype(np.float16).astype(np.float64))
    assert np.max(np.abs(got - exact)) <= 2.0 ** -11 * np.max(np.abs(exact)) + 2.0 ** -25
    # a power-of-two scale changes nothing but the exponent
    assert np.array_equal(oracle.dequantize_e4m3(bits, 0.25), oracle.e4m3_to_f64(bits) * 0.25)


def test_synthetic_quantiser_round_trips_within_half_an_e4m3_step():
    rng = np.random.default_rng(6)
    x = rng.standard_normal((3, 2, 128, 128)).astype(np.float32)
    bits, scale = inputs.quantize_e4m3_pages(x)
    assert bits.dtype == np.uint8 and scale.shape == (3, 2)
    deq = oracle.dequantize_e4m3(bits, scale[:, :, None, None])
    # e4m3 keeps 4 significant bits: relative error <= 2^-4 for normal values, absolute 2^-10 scale below
    assert np.all(np.abs(deq - x) <= 2.0 ** -4 * np.abs(x) + 2.0 ** -9 * scale[:, :, None, None] + 1e-3)
    assert np.abs(deq).max() <= 448 * scale.max() * 1.001
