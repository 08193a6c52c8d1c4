"""Pins for the zero-point dequantiser (paper Section II-B: uniform quantiser with a
zero-point, so w = step * (q - zero_point))."""
import numpy as np
import pytest
import torch

import oracle


@pytest.mark.parametrize("zp,scale", [(0, 1.0), (7, 0.02), (127, 0.1 / 256), (3, 0.05), (15, 1.0 / 3.0),
                                      (31, 3.0e-39), (1, 257.0 / 65536.0), (127, 1.0 + 2.0 ** -8)])
def test_against_library_conversions(zp, scale):
    """Exhaustive over all 256 symbols: fp32 result equals numpy's single-precision
    product; bf16 equals torch's float32 -> bfloat16 conversion (round to nearest even)."""
    sym = np.arange(256, dtype=np.uint8)
    f = oracle.dequant(sym, zp, scale, "f32")
    want = (sym.astype(np.int32) - zp).astype(np.float32) * np.float32(scale)
    assert f.dtype == np.float32 and (f.view(np.uint32) == want.view(np.uint32)).all()
    b = oracle.dequant(sym, zp, scale, "bf16")
    tb = torch.from_numpy(want).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (b == tb).all()


def test_bf16_ties_round_to_even():
    # (q - zp) * scale with scale = 1 + 2^-8: products k + k/256 have exact ties at the
    # bf16 boundary for suitable k; check a few by hand
    sym = np.array([1, 2, 3, 128, 129], dtype=np.uint8)
    scale = 1.0 + 2.0 ** -8          # 0x3F808000: exactly half way between two bf16 values
    b = oracle.dequant(sym, 0, scale, "bf16")
    assert b[0] == 0x3F80            # tie, kept mantissa even -> round down
    assert b[1] == 0x4000            # 2.0078125 = 0x40008000: tie, even -> down
    assert b[2] == 0x4041            # 3.01171875 = 0x4040C000: above half -> up
    s2 = 1.0 + 3 * 2.0 ** -8         # 0x3F818000: tie with odd kept lsb -> round up
    assert oracle.dequant(np.array([1], np.uint8), 0, s2, "bf16")[0] == 0x3F82


def test_zero_point_maps_to_zero_and_symmetry():
    sym = np.arange(15, dtype=np.uint8)
    f = oracle.dequant(sym, 7, 0.02, "f32")
    assert f[7] == 0.0 and np.allclose(f[:7][::-1], -f[8:])
    assert (oracle.dequant(sym, 7, 0.02, "u8") == sym).all()
