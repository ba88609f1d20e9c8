"""Pins for the oracle's quantised base weights (Sec. 5 names a quantised base model with 16-bit adapters as a
variant and fixes no format; the format taken is the 8-bit float with 4 exponent / 3 mantissa bits, bias 7, no
infinities, and one fp32 scale per output row).  External reference: torch's float8_e4m3fn conversion."""
import numpy as np
import torch

import moin_inputs as mi
import oracle


def test_all_256_codes_against_torch_float8():
    codes = torch.arange(256, dtype=torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = np.array([oracle.e4m3_value(c) for c in range(256)])
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan) and set(np.nonzero(nan)[0]) == {0x7F, 0xFF}
    assert np.array_equal(got[~nan], ref[~nan])
    # landmarks of the format: largest finite value, smallest subnormal, one, signed zero
    assert oracle.e4m3_value(0x7E) == 448.0 and oracle.e4m3_value(0x01) == 2.0 ** -9
    assert oracle.e4m3_value(0x38) == 1.0 and oracle.e4m3_value(0x80) == 0.0 and np.signbit(oracle.e4m3_value(0x80))


def test_dequantised_weight_against_torch_and_the_layer_on_it():
    rng = np.random.default_rng(3)
    d_out, d_in = 48, 64
    codes = rng.integers(0, 256, size=(d_out, d_in)).astype(np.uint8)
    codes[(codes & 0x7F) == 0x7F] = 0x3A                                  # no NaN codes in a weight matrix
    scale = np.exp(rng.uniform(-6, 1, size=d_out)).astype(np.float32)     # arbitrary positive scales, not powers of two
    bits = oracle.dequant_fp8(codes, scale)
    ref = (torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float32) * torch.from_numpy(scale)[:, None]).to(torch.bfloat16)
    assert np.array_equal(bits, mi.bf16_bits(ref))
    # power-of-two scales lose nothing: the weight is exactly value * scale
    s2 = (2.0 ** rng.integers(-8, 3, size=d_out)).astype(np.float32)
    w = mi.bf16_to_f64(torch.from_numpy(oracle.dequant_fp8(codes, s2).view(np.int16)).view(torch.bfloat16))
    vals = np.array([oracle.e4m3_value(c) for c in codes.ravel()]).reshape(codes.shape)
    assert np.array_equal(w, vals * s2[:, None].astype(np.float64))
    # the layer on a quantised base = the ordinary layer on the dequantised weight (numpy merged-weight identity)
    x = rng.normal(size=(9, d_in))
    A, B = rng.normal(size=(1, 4, d_in)) * 0.1, rng.normal(size=(1, d_out, 4)) * 0.1
    y = oracle.lora_linear(x, w, A, B, np.zeros(9, np.int32), np.zeros(1, np.int32), 2.0)
    np.testing.assert_allclose(y, x @ (w + 2.0 * B[0] @ A[0]).T, rtol=1e-12, atol=1e-12)
