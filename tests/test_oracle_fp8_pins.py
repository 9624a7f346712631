"""Pins of the E4M3-cache oracle: the 8-bit decoder against the format's landmark values and a library
conversion of every code; the attention against the (separately pinned) bf16 definition on the decoded values,
which is exact because every E4M3 value is a bf16 value; and the two scale identities."""
import math

import numpy as np
import pytest

from oracle import attention_oracle as O
from paper_2606_03077_b200 import workloads as W


def test_e4m3_landmarks():
    dec = O.e4m3_to_f64(np.arange(256, dtype=np.uint8))
    assert dec[0x00] == 0.0 and dec[0x80] == 0.0 and math.copysign(1.0, dec[0x80]) == -1.0
    assert dec[0x38] == 1.0 and dec[0xB8] == -1.0          # exponent field 7, mantissa 0
    assert dec[0x3C] == 1.5 and dec[0x40] == 2.0
    assert dec[0x01] == 2.0 ** -9                          # smallest subnormal
    assert dec[0x07] == 7 * 2.0 ** -9 and dec[0x08] == 2.0 ** -6   # largest subnormal, smallest normal
    assert dec[0x7E] == 448.0 and dec[0xFE] == -448.0      # largest finite
    assert np.isnan(dec[0x7F]) and np.isnan(dec[0xFF])
    assert np.sum(np.isnan(dec)) == 2 and not np.any(np.isinf(dec))
    pos = dec[:0x7F]
    assert np.all(np.diff(pos) > 0)                        # codes order like magnitudes
    assert np.array_equal(dec[0x80:0xFF], -pos)


def test_e4m3_matches_library_conversion_of_all_codes():
    torch = pytest.importorskip("torch")
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("no float8 type in this torch")
    codes = torch.arange(256, dtype=torch.int16).to(torch.uint8)
    lib = codes.view(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    dec = O.e4m3_to_f64(codes.numpy())
    assert np.array_equal(np.isnan(lib), np.isnan(dec))
    ok = ~np.isnan(dec)
    assert np.array_equal(lib[ok], dec[ok])


def decoded_as_bf16_bits(codes):
    """E4M3 codes -> bf16 bit patterns of the same values, by the library (torch) route."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(codes)).view(torch.float8_e4m3fn).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def test_equals_bf16_definition_on_decoded_values():
    pytest.importorskip("torch")
    lens, bt, q, k8, v8 = W.random_case_e4m3(21, 4, 8, 2, 32, (1, 17, 40, 0), poison=False)
    out8, lse8 = O.paged_decode_attention_fp8(q, k8, v8, bt, lens)
    out16, lse16 = O.paged_decode_attention(q, decoded_as_bf16_bits(k8), decoded_as_bf16_bits(v8), bt, lens)
    assert np.array_equal(out8[:3], out16[:3]) and np.array_equal(lse8[:3], lse16[:3])
    assert np.all(out8[3] == 0) and np.all(np.isneginf(lse8[3]))


def test_scale_identities():
    pytest.importorskip("torch")
    lens, bt, q, k8, v8 = W.random_case_e4m3(22, 3, 4, 2, 16, (5, 33, 64), poison=False)
    base, lse0 = O.paged_decode_attention_fp8(q, k8, v8, bt, lens)
    # the value scale multiplies the output and leaves lse alone
    out, lse = O.paged_decode_attention_fp8(q, k8, v8, bt, lens, v_scale=0.375)
    assert np.allclose(out, 0.375 * base, rtol=1e-13, atol=0) and np.array_equal(lse, lse0)
    out, _ = O.paged_decode_attention_fp8(q, k8, v8, bt, lens, v_scale=0.25)   # a power of two: exact
    assert np.array_equal(out, 0.25 * base)
    # the key scale is a softmax scale: same as the bf16 definition with sm_scale * k_scale
    ks = 0.6
    out, lse = O.paged_decode_attention_fp8(q, k8, v8, bt, lens, k_scale=ks)
    ref, lref = O.paged_decode_attention(q, decoded_as_bf16_bits(k8), decoded_as_bf16_bits(v8), bt, lens,
                                         sm_scale=ks / math.sqrt(16))
    assert np.allclose(out, ref, rtol=0, atol=1e-13) and np.allclose(lse, lref, rtol=0, atol=1e-12)


def test_nan_codes_outside_sequences_are_never_read():
    lens, bt, q, k8, v8 = W.random_case_e4m3(23, 3, 4, 1, 16, (3, 16, 21))
    assert np.any(k8 == W.E4M3_NAN)
    out, lse = O.paged_decode_attention_fp8(q, k8, v8, bt, lens)
    assert np.all(np.isfinite(out)) and np.all(np.isfinite(lse))


def test_length_one_returns_the_scaled_value_row():
    lens, bt, q, k8, v8 = W.random_case_e4m3(24, 2, 4, 2, 16, (1, 1))
    out, _ = O.paged_decode_attention_fp8(q, k8, v8, bt, lens, k_scale=3.0, v_scale=0.25)
    for b in range(2):
        for h in range(4):
            want = 0.25 * O.e4m3_to_f64(v8[bt[b, 0], h // 2, 0])
            assert np.array_equal(out[b, h], want)
