"""Pins of the oracle's physical layout rule (bijection, hand-worked positions)."""

import numpy as np
import pytest

import oracle


def test_packed_sizes():
    assert oracle.packed_sizes(4096, 4096) == (4096 * 4096 // 2, 32 * 4096 * 4)
    assert oracle.packed_sizes(13696, 4096) == (13696 * 4096 // 2, 107 * 4096 * 4)
    with pytest.raises(ValueError):
        oracle.packed_sizes(100, 16)
    with pytest.raises(ValueError):
        oracle.packed_sizes(128, 24)


def test_pack_is_a_bijection_and_unpack_inverts_it():
    rng = np.random.default_rng(0)
    K, N = 384, 176
    codes = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    d = rng.standard_normal((K // 128, N)).astype(np.float16)
    b = oracle.e0m4_value(rng.integers(0, 16, size=(K // 128, N)))
    packed, scales = oracle.pack(codes, d, b)
    assert packed.nbytes == K * N // 2 and scales.nbytes == (K // 128) * N * 4
    c2, d2, b2 = oracle.unpack(packed, scales, K, N)
    assert np.array_equal(c2, codes)
    assert np.array_equal(d2.view(np.uint16), d.view(np.uint16))
    assert np.array_equal(b2.view(np.uint16), b.view(np.uint16))
    # every nibble is written exactly once: all-ones codes fill every bit
    full, _ = oracle.pack(np.full((K, N), 15, np.uint8), d, b)
    assert np.all(full == 0xFFFFFFFF)


def test_single_code_lands_where_the_rule_says():
    # Worked by hand from the layout rule in include/tl_e0m4.h, K = 256 (2 groups), N = 160
    # (panel 0 holds 8 column blocks, panel 1 the remaining 2):
    #   (k, n) = (0, 0)      -> tile 0, word 0, nibble 0
    #   (k, n) = (1, 0)      -> word 0, nibble 4                  (odd k -> high half)
    #   (k, n) = (6, 0)      -> word 0, nibble 3
    #   (k, n) = (9, 3)      -> tile 0, column 3 -> word 3*16 + 1 = 49, nibble 4
    #   (k, n) = (130, 17)   -> panel 0, g = 1, r = 1 -> tile 1*8 + 1 = 9
    #                           -> word 9*256 + 1*16 + 0 = 2320, nibble 1
    #   (k, n) = (5, 150)    -> panel 1 (R = 2) starts at tile 16; g = 0, r = 1 -> tile 17
    #                           -> word 17*256 + 6*16 + 0 = 4448, nibble 2 + 4 = 6
    #   (k, n) = (128, 130)  -> panel 1, g = 1, r = 0 -> tile 16 + 1*2 + 0 = 18
    #                           -> word 18*256 + 2*16 + 0 = 4640, nibble 0
    cases = [((0, 0), 0, 0), ((1, 0), 0, 4), ((6, 0), 0, 3), ((9, 3), 49, 4),
             ((130, 17), 2320, 1), ((5, 150), 4448, 6), ((128, 130), 4640, 0)]
    K, N = 256, 160
    zeros = np.zeros((K // 128, N), np.float16)
    for (k, n), word, nib in cases:
        codes = np.zeros((K, N), np.uint8)
        codes[k, n] = 0xB
        packed, _ = oracle.pack(codes, zeros, zeros)
        assert packed[word] == np.uint32(0xB << (4 * nib)), (k, n)
        assert np.count_nonzero(packed) == 1


def test_scale_word_position_and_halves():
    K, N = 256, 160
    d = np.zeros((2, N), np.float16)
    b = np.zeros((2, N), np.float16)
    d[1, 17] = np.float16(0.5)    # bits 0x3800
    b[1, 17] = np.float16(2.375)  # bits 0x40C0
    d[0, 150] = np.float16(1.0)   # bits 0x3C00
    _, scales = oracle.pack(np.zeros((K, N), np.uint8), d, b)
    # (g=1, n=17) -> tile 9, column 1 -> word 9*16 + 1; (g=0, n=150) -> tile 17, column 6
    assert scales[9 * 16 + 1] == np.uint32(0x40C03800)
    assert scales[17 * 16 + 6] == np.uint32(0x00003C00)
    assert np.count_nonzero(scales) == 2


@pytest.mark.parametrize("group", [32, 64])
def test_smaller_groups_pack_and_unpack(group):
    rng = np.random.default_rng(group)
    K, N = 384, 176
    ng = K // group
    codes = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    d = rng.standard_normal((ng, N)).astype(np.float16)
    b = oracle.e0m4_value(rng.integers(0, 16, size=(ng, N)))
    packed, scales = oracle.pack(codes, d, b, group)
    assert (packed.nbytes, scales.nbytes) == oracle.packed_sizes(K, N, group) == (K * N // 2, ng * N * 4)
    # the codes do not move with the group size
    assert np.array_equal(packed, oracle.pack(codes, d[: K // 128], b[: K // 128])[0])
    c2, d2, b2 = oracle.unpack(packed, scales, K, N, group)
    assert np.array_equal(c2, codes)
    assert np.array_equal(d2.view(np.uint16), d.view(np.uint16))
    assert np.array_equal(b2.view(np.uint16), b.view(np.uint16))
    # every coefficient word is written exactly once
    ones = np.full((ng, N), np.float16(1.0))
    _, full = oracle.pack(codes, ones, ones, group)
    assert np.all(full == 0x3C003C00)


def test_scale_word_position_with_smaller_groups():
    # Worked by hand, K = 256, N = 160 as above.  G = 32 (4 runs of 16 words per tile):
    #   (k group 5 = rows 160..191, n = 17): tile row g = 1, r = 1 -> tile 9; run (160 % 128) // 32 = 1
    #       -> word (9*4 + 1)*16 + 1 = 593
    #   (k group 3 = rows 96..127, n = 150): panel 1 starts at tile 16, g = 0, r = 1 -> tile 17; run 3
    #       -> word (17*4 + 3)*16 + 6 = 1142
    # G = 64 (2 runs): (k group 3 = rows 192..255, n = 130): tile 16 + 1*2 + 0 = 18; run 1
    #       -> word (18*2 + 1)*16 + 2 = 594
    K, N = 256, 160
    d = np.zeros((8, N), np.float16)
    b = np.zeros((8, N), np.float16)
    d[5, 17] = np.float16(0.5)
    b[5, 17] = np.float16(2.375)
    d[3, 150] = np.float16(1.0)
    _, scales = oracle.pack(np.zeros((K, N), np.uint8), d, b, 32)
    assert scales[593] == np.uint32(0x40C03800)
    assert scales[1142] == np.uint32(0x00003C00)
    assert np.count_nonzero(scales) == 2
    d = np.zeros((4, N), np.float16)
    d[3, 130] = np.float16(2.0)  # bits 0x4000
    _, scales = oracle.pack(np.zeros((K, N), np.uint8), d, d * 0, 64)
    assert scales[594] == np.uint32(0x00004000)
    assert np.count_nonzero(scales) == 1


# ------------------------------------------------------------------ 3-bit and 5-bit codes
@pytest.mark.parametrize("bits", [3, 5])
def test_odd_width_pack_is_a_bijection(bits):
    rng = np.random.default_rng(bits)
    K, N = 384, 176
    codes = rng.integers(0, 1 << bits, size=(K, N), dtype=np.uint8)
    d = rng.standard_normal((K // 128, N)).astype(np.float16)
    b = oracle.e0m4_value(rng.integers(0, 1 << bits, size=(K // 128, N)), bits=bits)
    packed, scales = oracle.pack(codes, d, b, bits=bits)
    assert packed.nbytes == K * N * bits // 8 == oracle.packed_sizes(K, N, bits=bits)[0]
    c2, d2, b2 = oracle.unpack(packed, scales, K, N, bits=bits)
    assert np.array_equal(c2, codes)
    assert np.array_equal(d2.view(np.uint16), d.view(np.uint16))
    assert np.array_equal(b2.view(np.uint16), b.view(np.uint16))
    # every bit is written exactly once: all-ones codes fill every bit of the stream
    full, _ = oracle.pack(np.full((K, N), (1 << bits) - 1, np.uint8), d, b, bits=bits)
    assert np.all(full == 0xFFFFFFFF)
    # the coefficient words are those of the 4-bit container
    assert np.array_equal(scales, oracle.pack(np.zeros((K, N), np.uint8), d, b)[1])


def test_odd_width_codes_land_where_the_rule_says():
    # Worked by hand, K = 256 (2 groups), N = 160 (panel 0: 8 column blocks, panel 1: 2), code = all ones.
    # 5 bits: a tile is 1280 bytes, a column owns 80 of them, a unit of eight k is 5 bytes.
    #   (k, n) = (0, 0)     -> bit 0                      -> byte 0, bits 0..4
    #   (k, n) = (1, 0)     -> bit 5                      -> byte 0 bits 5..7 and byte 1 bits 0..1
    #   (k, n) = (7, 0)     -> bit 35                     -> byte 4 bits 3..7 (the unit's last byte)
    #   (k, n) = (8, 0)     -> bit 40                     -> byte 5 bits 0..4 (next unit)
    #   (k, n) = (9, 3)     -> column 3 starts at byte 240; bit 45 of it -> byte 245 bits 5..7, byte 246 bits 0..1
    #   (k, n) = (130, 17)  -> tile 9 (see the 4-bit test) at byte 11520, column 1 at +80; k % 128 = 2 -> bit 10
    #                          -> byte 11601 bits 2..6
    #   (k, n) = (128, 130) -> tile 18 at byte 23040, column 2 at +160, bit 0 -> byte 23200 bits 0..4
    cases5 = [((0, 0), {0: 0x1F}), ((1, 0), {0: 0xE0, 1: 0x03}), ((7, 0), {4: 0xF8}), ((8, 0), {5: 0x1F}),
              ((9, 3), {245: 0xE0, 246: 0x03}), ((130, 17), {11601: 0x7C}), ((128, 130), {23200: 0x1F})]
    # 3 bits: a tile is 768 bytes, a column owns 48, a unit is 3 bytes.
    #   (k, n) = (2, 0)     -> bit 6   -> byte 0 bits 6..7 and byte 1 bit 0
    #   (k, n) = (7, 0)     -> bit 21  -> byte 2 bits 5..7
    #   (k, n) = (9, 3)     -> column 3 at byte 144; bit 27 -> byte 147 bits 3..5
    #   (k, n) = (130, 17)  -> tile 9 at byte 6912, column 1 at +48; bit 6 -> byte 6960 bits 6..7, byte 6961 bit 0
    cases3 = [((2, 0), {0: 0xC0, 1: 0x01}), ((7, 0), {2: 0xE0}), ((9, 3), {147: 0x38}),
              ((130, 17), {6960: 0xC0, 6961: 0x01})]
    K, N = 256, 160
    zeros = np.zeros((K // 128, N), np.float16)
    for bits, cases in ((5, cases5), (3, cases3)):
        for (k, n), expect in cases:
            codes = np.zeros((K, N), np.uint8)
            codes[k, n] = (1 << bits) - 1
            packed, _ = oracle.pack(codes, zeros, zeros, bits=bits)
            stream = packed.astype("<u4").view(np.uint8)
            assert {int(i): int(stream[i]) for i in np.flatnonzero(stream)} == expect, (bits, k, n)


def test_odd_width_code_value_sits_low_bit_first():
    # code 0b10110 (22) at (k, n) = (1, 0): bits 5..9 of the stream = 0,1,1,0,1 -> byte 0 = 0b110_00000, byte 1 = 0b10
    codes = np.zeros((128, 16), np.uint8)
    codes[1, 0] = 0b10110
    zeros = np.zeros((1, 16), np.float16)
    stream = oracle.pack(codes, zeros, zeros, bits=5)[0].astype("<u4").view(np.uint8)
    assert stream[0] == 0b11000000 and stream[1] == 0b00000010 and not stream[2:].any()
