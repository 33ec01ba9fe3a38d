"""Physical layout of the packed E0M4 weights (test infrastructure only).

The paper gives no storage layout (Section 2.3 only says the codes are 4-bit
and the coefficients are per group), so the layout is this library's own rule.
It is restated here independently of the CUDA packer so that packed bytes can
be compared bit for bit:

  tile   : 16 columns x 128 rows (one group) of codes = 256 uint32 words.
  panel  : up to 8 neighbouring tiles (128 columns); panel p = n // 128 holds
           R = min(8, N/16 - 8p) column blocks.  Panels are stored one after
           the other; inside a panel the tiles are ordered group by group:
           tile number = p * 8 * (K/128) + g * R + r,   g = k // 128,
           r = (n % 128) // 16.
  packed : uint32 words, tile after tile.  Inside a tile, column n % 16 owns 16
           consecutive words; word (k % 128) // 8 holds eight consecutive k; the
           code of k_local = k % 8 sits in nibble k_local // 2 + 4 * (k_local % 2)
           (bits 4p .. 4p+3), so the low and the high 16-bit halves carry the
           even and the odd k of each pair at the same nibble position.
  scales : uint32 words, 16 per tile in the same tile order (word = tile * 16 +
           n % 16): low half = fp16 bits of the dequantization scale d, high
           half = fp16 bits of the bias b.
           Group sizes 64 and 32 keep the tile of 128 rows; a tile then owns
           128/G runs of 16 words, one per group of its rows:
           word = (tile * (128/G) + (k % 128) // G) * 16 + n % 16.

8-bit codes (``bits=8``): the same tiles in the same order, one byte per code, so a tile is
2048 bytes, made of eight chunks of 256 bytes, one per 16 rows; in chunk (k % 128) // 16 column
n % 16 owns 16 consecutive bytes and byte k % 16 of them is the code of row k.  The
coefficient words do not change.

3-bit and 5-bit codes (``bits=3``, ``bits=5``): the same tiles in the same order.  Eight
consecutive k of one column form a unit of ``bits`` bytes, read as a little-endian integer in
which the code of k % 8 = c occupies bits c * bits .. (c + 1) * bits - 1.  Inside a tile column
n % 16 owns its 16 units one after the other (16 * bits bytes), so a tile is 256 * bits bytes and
the 128 codes of a column's tile row are one continuous little-endian bit string: the code of row
k starts at bit (k % 128) * bits of it.  The coefficient words do not change.
"""

from __future__ import annotations

import numpy as np

TILE_N = 16
TILE_K = 128
PANEL_TILES = 8


def packed_sizes(K: int, N: int, group: int = TILE_K, bits: int = 4):
    """Bytes of the packed-code buffer and of the coefficient buffer."""
    if bits not in (3, 4, 5, 8):
        raise ValueError("the container holds 3-, 4-, 5- or 8-bit codes")
    if K <= 0 or N <= 0 or K % TILE_K or N % TILE_N:
        raise ValueError("K must be a multiple of 128 and N a multiple of 16")
    if group not in (32, 64, 128):
        raise ValueError("group must be 32, 64 or 128")
    return K * N * bits // 8, (K // group) * N * 4


def _nibble_pos(k_local):
    return k_local // 2 + 4 * (k_local % 2)


def _tile_index(k, n, K, N):
    ng = K // TILE_K
    nb = n // TILE_N
    p = nb // PANEL_TILES
    r = nb % PANEL_TILES
    R = np.minimum(PANEL_TILES, N // TILE_N - PANEL_TILES * p)
    return p * PANEL_TILES * ng + (k // TILE_K) * R + r


def _scale_word(K, N, group):
    """Index of the coefficient word of every (group, column): [K/G, N]."""
    subs = TILE_K // group
    kg = (np.arange(K // group) * group)[:, None]
    n = np.arange(N)[None, :]
    return (_tile_index(kg, n, K, N) * subs + (kg % TILE_K) // group) * 16 + (n % TILE_N)


def _byte_index(K, N):
    """Position of every 8-bit code in the packed byte stream: [K, N]."""
    k = np.arange(K)[:, None]
    n = np.arange(N)[None, :]
    chunk = (k % TILE_K) // 16
    return _tile_index(k, n, K, N) * (TILE_N * TILE_K) + chunk * (TILE_N * 16) + (n % TILE_N) * 16 + k % 16


def _bit_index(K, N, bits):
    """Position (in bits from the start of the packed stream) of the lowest bit of every 3- or
    5-bit code: [K, N]."""
    k = np.arange(K)[:, None]
    n = np.arange(N)[None, :]
    column_start = _tile_index(k, n, K, N) * (256 * bits) + (n % TILE_N) * (16 * bits)  # bytes
    return column_start * 8 + (k % TILE_K) * bits


def pack(codes, d_h, b_h, group: int = TILE_K, bits: int = 4):
    """Logical (codes[K,N] uint8, d_h[K/G,N] fp16, b_h[K/G,N] fp16) ->
    (packed uint32[K*N*bits/32], scales uint32[K/G*N])."""
    codes = np.asarray(codes, dtype=np.uint8)
    K, N = codes.shape
    packed_sizes(K, N, group, bits)
    ng = K // group
    k = np.arange(K)[:, None]
    n = np.arange(N)[None, :]
    if bits == 8:
        stream = np.zeros(K * N, dtype=np.uint8)
        stream[_byte_index(K, N).ravel()] = codes.ravel()
        packed = stream.view("<u4").astype(np.uint32)
    elif bits in (3, 5):
        # one bit at a time into a stream of single bits, then eight bits to the byte, lowest first
        stream_bits = np.zeros(K * N * bits, dtype=np.uint8)
        start = _bit_index(K, N, bits).ravel()
        flat = codes.ravel()
        for i in range(bits):
            stream_bits[start + i] = (flat >> i) & 1
        packed = np.packbits(stream_bits, bitorder="little").view("<u4").astype(np.uint32)
    else:
        word = _tile_index(k, n, K, N) * 256 + (n % TILE_N) * 16 + (k % TILE_K) // 8
        shift = (4 * _nibble_pos(k % 8)).astype(np.uint32) + np.zeros_like(n, dtype=np.uint32)
        packed = np.zeros(K * N // 8, dtype=np.uint32)
        np.bitwise_or.at(packed, word.ravel(), (codes.astype(np.uint32) << shift).ravel())

    sword = _scale_word(K, N, group)
    d_bits = np.asarray(d_h, dtype=np.float16).view(np.uint16).astype(np.uint32)
    b_bits = np.asarray(b_h, dtype=np.float16).view(np.uint16).astype(np.uint32)
    scales = np.zeros(ng * N, dtype=np.uint32)
    scales[sword.ravel()] = (d_bits | (b_bits << np.uint32(16))).ravel()
    return packed, scales


def unpack(packed, scales, K: int, N: int, group: int = TILE_K, bits: int = 4):
    """Inverse of pack()."""
    packed = np.asarray(packed).view(np.uint32).ravel()
    scales = np.asarray(scales).view(np.uint32).ravel()
    packed_sizes(K, N, group, bits)
    k = np.arange(K)[:, None]
    n = np.arange(N)[None, :]
    if bits == 8:
        codes = packed.astype("<u4").view(np.uint8)[_byte_index(K, N)]
    elif bits in (3, 5):
        stream_bits = np.unpackbits(packed.astype("<u4").view(np.uint8), bitorder="little")
        start = _bit_index(K, N, bits)
        codes = np.zeros((K, N), dtype=np.uint8)
        for i in range(bits):
            codes |= (stream_bits[start + i] << i).astype(np.uint8)
    else:
        word = _tile_index(k, n, K, N) * 256 + (n % TILE_N) * 16 + (k % TILE_K) // 8
        shift = (4 * _nibble_pos(k % 8)).astype(np.uint32) + np.zeros_like(n, dtype=np.uint32)
        codes = ((packed[word] >> shift) & np.uint32(0xF)).astype(np.uint8)
    s = scales[_scale_word(K, N, group)]
    d_h = (s & np.uint32(0xFFFF)).astype(np.uint16).view(np.float16)
    b_h = (s >> np.uint32(16)).astype(np.uint16).view(np.float16)
    return codes, d_h, b_h
