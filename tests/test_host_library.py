"""Host-side checks of the C-ABI library: it loads, exports every symbol include/lcd.h declares, the packer is
bit-identical to the oracle's and invalid arguments come back as status codes (no compute calls here)."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2506_12038_b200 as lcd
from paper_2506_12038_b200 import binding
from oracle import lcd_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "lcd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lcd_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 10
    dll = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(dll, n), n
    assert sorted(binding.EXPORTS) == names


@pytest.mark.parametrize("bits,C,N,K", [(2, 4, 19, 700), (3, 8, 19, 700), (3, 5, 8, 256), (2, 3, 1, 1), (2, 4, 64, 1024),
                                       (3, 8, 33, 513), (4, 16, 19, 700), (4, 10, 33, 513), (4, 9, 1, 1)])
def test_packer_matches_oracle_bit_for_bit(bits, C, N, K):
    rng = np.random.default_rng(N * 1000 + K + bits)
    idx = rng.integers(0, C, size=(N, K), dtype=np.uint8)
    cb = rng.standard_normal((N, C)).astype(np.float16)
    blob = lcd.pack_weights(idx, cb, bits, C)
    assert blob.size == lcd.packed_weights_bytes(N, K, bits) == O.packed_weights_bytes(N, K, bits)
    assert np.array_equal(blob, O.pack_weights(idx, cb, bits, C))
    # cross round trips: library unpack of oracle blob, oracle unpack of library blob
    i2, c2, b2, C2 = lcd.unpack_weights(O.pack_weights(idx, cb, bits, C))
    assert np.array_equal(i2, idx) and np.array_equal(c2.view(np.uint16), cb.view(np.uint16)) and (b2, C2) == (bits, C)
    i3, c3, _, _ = O.unpack_weights(blob)
    assert np.array_equal(i3, idx) and np.array_equal(c3.view(np.uint16), cb.view(np.uint16))


def test_packer_edge_patterns():
    for bits in (2, 3, 4):
        C = 1 << bits
        cb = np.zeros((8, C), dtype=np.float16)
        for fill in (0, C - 1):
            idx = np.full((8, 256), fill, dtype=np.uint8)
            assert np.array_equal(lcd.pack_weights(idx, cb, bits), O.pack_weights(idx, cb, bits))


def test_packer_error_codes():
    idx = np.zeros((4, 8), dtype=np.uint8)
    cb = np.zeros((4, 3), dtype=np.float16)
    idx[2, 5] = 3
    with pytest.raises(lcd.LcdError) as e:
        lcd.pack_weights(idx, cb, 2, 3)
    assert e.value.status == 4 and "n=2 k=5" in str(e.value)
    with pytest.raises(lcd.LcdError) as e:
        lcd.pack_weights(np.zeros((4, 8), dtype=np.uint8), np.zeros((4, 32), dtype=np.float16), 5, 32)
    assert e.value.status == 2        # five-bit indices: no kernel
    lib = binding.lib
    out = ctypes.c_size_t()
    assert lib.lcd_packed_weights_bytes(0, 8, 2, ctypes.byref(out)) == 1
    assert lib.lcd_packed_weights_bytes(8, 8, 2, None) == 1
    good = lcd.pack_weights(np.zeros((4, 8), dtype=np.uint8), cb, 2, 3)
    small = np.empty(good.size - 1, dtype=np.uint8)
    st = lib.lcd_pack_weights(np.zeros((4, 8), dtype=np.uint8).ctypes.data, cb.ctypes.data, 4, 8, 2, 3,
                              small.ctypes.data, small.size, None, None)
    assert st == 3
    for pos in (0, 4, 40, 300, good.size - 1):
        bad = good.copy()
        bad[pos] ^= 0x10
        with pytest.raises(lcd.LcdError) as e:
            lcd.unpack_weights(bad)
        assert e.value.status == 5
    with pytest.raises(lcd.LcdError):
        lcd.unpack_weights(good[:100])
    assert lib.lcd_status_string(5).decode() == "bad packed-weights blob"


def test_device_entry_points_reject_bad_arguments_before_any_launch():
    lib = binding.lib
    hdr = ctypes.create_string_buffer(bytes(lcd.pack_weights(np.zeros((8, 256), dtype=np.uint8),
                                                             np.zeros((8, 4), dtype=np.float16), 2)[:64]), 64)
    out = ctypes.c_size_t()
    assert lib.lcd_lut_linear_workspace_bytes(hdr, 1, 0, ctypes.byref(out)) == 0
    assert lib.lcd_lut_linear_workspace_bytes(hdr, 0, 0, ctypes.byref(out)) == 1
    assert lib.lcd_lut_linear_workspace_bytes(ctypes.create_string_buffer(64), 1, 0, ctypes.byref(out)) == 5
    assert lib.lcd_lut_linear(None, hdr, None, None, 1, None, 8, 0, None, 0, None, None) == 1
    assert lib.lcd_smooth_quantize_act(None, 1, 8, 8, None, None, 4, None, None, None) == 1
    fake = ctypes.c_void_p(4096)
    assert lib.lcd_smooth_quantize_act(fake, 1, 8, 4, None, None, 4, fake, fake, None) == 1      # ldx < K
    assert lib.lcd_smooth_quantize_act(fake, 1, 8, 8, None, None, 5, fake, fake, None) == 2      # act_bits: 4 or 8
    assert lib.lcd_lut_linear_act8(None, hdr, None, None, 1, None, 8, 0, None, 0, None, None) == 1
    assert lib.lcd_lut_linear(fake, hdr, fake, fake, 1, fake, 4, 0, None, 0, None, None) == 1     # ldy < N
    assert lib.lcd_lut_linear(ctypes.c_void_p(4100), hdr, fake, fake, 1, fake, 8, 1, None, 0, None, None) == 1
    assert lib.lcd_lut_linear(fake, hdr, fake, fake, 17, fake, 8, 3, None, 0, None, None) == 2    # M > 16
    assert lib.lcd_linear_host(fake, hdr, fake, 1, None, fake, fake, 16, None, None) == 3         # scratch small


def test_every_export_declares_its_argument_types():
    # an undeclared prototype makes ctypes pass Python ints as 32-bit values: 64-bit sizes and strides arrive wrong
    from paper_2506_12038_b200 import binding
    for name in binding.EXPORTS:
        if name != "lcd_last_cuda_error":
            assert getattr(binding.lib, name).argtypes, name
