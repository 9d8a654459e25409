"""Pins of the oracle's base-3 packed layout (five ternary codes per byte, 1.6 bits per weight: the
nearest byte-aligned packing to the paper's 1.58 bits) against its written description: round trips,
worked positions, the bijection between weights and (byte, digit) places, tile order and padding."""
import numpy as np

import oracle


def test_size_is_one_fifth_of_the_padded_matrix():
    assert oracle.packed_bytes_b3(16, 320) == 1024
    assert oracle.packed_bytes_b3(17, 321) == 32 * 640 // 5
    assert oracle.packed_bytes_b3(4096, 4096) == 4096 * 4160 // 5          # 1.625 bits per weight with the padding
    assert oracle.packed_bytes_b3(3200, 3200) * 8 / (3200 * 3200) == 1.6


def test_round_trip_random_and_constant():
    rng = np.random.default_rng(41)
    for shape in [(16, 320), (40, 704), (7, 64), (33, 1024)]:
        T = rng.integers(-1, 2, size=shape, dtype=np.int8)
        packed = oracle.pack_b3(T)
        assert packed.max() <= 242
        back, bad = oracle.unpack_b3(packed, *shape, return_bad=True)
        assert bad == 0 and np.array_equal(back, T)
    for v, byte in ((-1, 0), (0, 121), (1, 242)):                          # 121 = 1 + 3 + 9 + 27 + 81
        T = np.full((16, 320), v, np.int8)
        assert np.all(oracle.pack_b3(T) == byte)


def test_worked_positions_of_the_written_description():
    # (row, column) -> (byte index inside the tile, power of three), worked by hand from the description:
    # column = 32 (p / 2) + 16 (p % 2) + 4 t + e;  p < 16: byte 16 t + p, digit e;  p >= 16: byte
    # 16 t + 4 (p - 16) + e, digit 4
    cases = {(0, 0): (0, 1), (0, 5): (16, 3), (0, 16): (1, 1), (0, 3): (0, 27), (0, 47): (16 * 3 + 2, 27),
             (0, 256): (0, 81), (0, 257): (1, 81), (0, 260): (16, 81), (0, 288): (8, 81), (0, 319): (63, 81),
             (5, 0): (5 * 64, 1), (15, 319): (15 * 64 + 63, 81)}
    zero = oracle.pack_b3(np.zeros((16, 320), np.int8)).astype(int)
    for (n, k), (byte, power) in cases.items():
        T = np.zeros((16, 320), np.int8)
        T[n, k] = 1
        diff = oracle.pack_b3(T).astype(int) - zero
        assert np.flatnonzero(diff).tolist() == [byte] and diff[byte] == power, (n, k)
        T[n, k] = -1
        diff = oracle.pack_b3(T).astype(int) - zero
        assert diff[byte] == -power


def test_every_weight_has_its_own_digit():
    zero = oracle.pack_b3(np.zeros((16, 320), np.int8)).astype(int)
    seen = set()
    T = np.zeros((16, 320), np.int8)
    for n in (0, 9):
        for k in range(320):
            T[n, k] = 1
            diff = oracle.pack_b3(T).astype(int) - zero
            T[n, k] = 0
            (byte,) = np.flatnonzero(diff)
            assert diff[byte] in (1, 3, 9, 27, 81) and n * 64 <= byte < (n + 1) * 64
            seen.add((int(byte), int(diff[byte])))
    assert len(seen) == 2 * 320                                             # 64 bytes x 5 digits per row, each used once


def test_tile_order_and_padding():
    T = np.zeros((32, 640), np.int8)
    T[0, 320] = 1          # tile (0, 1)
    T[16, 0] = 1           # tile (1, 0)
    p = oracle.pack_b3(T).astype(int)
    assert p[1024] == 122 and p[2048] == 122 and (p != 121).sum() == 2     # column tiles run fastest
    # ragged sizes: padding rows and columns decode as zero weights and do not disturb their neighbours
    rng = np.random.default_rng(42)
    T = rng.integers(-1, 2, size=(5, 128), dtype=np.int8)
    packed = oracle.pack_b3(T)
    assert packed.size == 1024
    full = oracle.unpack_b3(np.concatenate([packed]), 16, 320)
    assert np.array_equal(full[:5, :128], T) and not full[5:].any() and not full[:, 128:].any()


def test_invalid_bytes_are_reported():
    packed = oracle.pack_b3(np.zeros((16, 320), np.int8))
    packed[3] = 250
    T, bad = oracle.unpack_b3(packed, 16, 320, return_bad=True)
    assert bad == 1 and not T.any()
