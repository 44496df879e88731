"""Storage helpers of the input module (CPU only)."""
import numpy as np

from paper_2208_00763_b200 import inputs


def test_dense_storage_layout():
    rng = np.random.default_rng(0)
    bits1 = rng.integers(0, 2, 37)
    assert np.array_equal(inputs.to_dense(bits1, 1), np.packbits(bits1.astype(np.uint8), bitorder="little"))
    # signed 1-bit codes {-1, 0} store the same bit pattern as {1, 0}
    assert np.array_equal(inputs.to_dense(-bits1, 1), inputs.to_dense(bits1, 1))
    v4 = np.array([1, -1, 7, -8, 3])
    assert inputs.to_dense(v4, 4).tolist() == [0xF1, 0x87, 0x03]          # low nibble first, two's complement
    v2 = np.array([1, 2, 3, 0, -1, -2])
    assert inputs.to_dense(v2, 2).tolist() == [0b00111001, 0b00001011]
    v8 = rng.integers(-128, 128, 10)
    assert np.array_equal(inputs.to_dense(v8, 8).view(np.int8), v8.astype(np.int8))


def test_dense_round_trip_and_bit_order():
    import numpy as np
    from paper_2208_00763_b200 import inputs
    rng = np.random.default_rng(3)
    for bits in (1, 2, 4, 8):
        for signed in (False, True):
            lo, hi = inputs.code_range(bits, signed)
            v = rng.integers(lo, hi + 1, 1001)
            assert np.array_equal(inputs.from_dense(inputs.to_dense(v, bits), v.size, bits, signed), v)
    # written out by hand: 4-bit codes (1, -2, 7) -> bytes 0xE1, 0x07
    assert inputs.to_dense(np.array([1, -2, 7]), 4).tolist() == [0xE1, 0x07]
    assert inputs.from_dense(np.array([0xE1, 0x07], dtype=np.uint8), 3, 4, True).tolist() == [1, -2, 7]
    # 1-bit codes agree with numpy's little-endian bit packing
    b = rng.integers(0, 2, 77)
    assert np.array_equal(inputs.from_dense(np.packbits(b.astype(np.uint8), bitorder="little"), 77, 1, False), b)
