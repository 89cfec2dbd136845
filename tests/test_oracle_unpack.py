"""Pins for the oracle's decoders: hand-worked words, exhaustive nibbles, bf16 bit patterns."""
import numpy as np
import pytest

from oracle import tilefuse_oracle as orc
from paper_2606_11357_b200 import workloads as wl
from helpers import loop_pack_awq, read_golden_words


@pytest.mark.parametrize("codes,word", read_golden_words())
def test_golden_word_decodes(codes, word):
    got = orc.unpack_awq(np.array([[word]], dtype=np.uint32))
    assert got.dtype == np.uint8 and got.tolist() == [codes]


@pytest.mark.parametrize("codes,word", read_golden_words())
def test_golden_word_encodes(codes, word):
    """The input generator's encoder and the test-local loop encoder both hit the worked value."""
    arr = np.array([codes], dtype=np.uint8)
    assert int(wl.awq_pack_words(arr)[0, 0]) == word
    assert int(loop_pack_awq([codes])[0, 0]) == word


def test_adjacent_pair_property():
    """Masking a word with 0x000F000F yields an adjacent column pair: the reason for the order."""
    word = 0x75316420                       # columns 0..7 hold codes 0..7
    for shift, pair in enumerate([(0, 1), (2, 3), (4, 5), (6, 7)]):
        v = (word >> (4 * shift)) & 0x000F000F
        assert (v & 0xFFFF, v >> 16) == pair


def test_exhaustive_value_times_position():
    for column in range(8):
        for value in range(16):
            codes = [0] * 8
            codes[column] = value
            word = loop_pack_awq([codes])
            assert orc.unpack_awq(word).tolist() == [codes]


def test_unpack_matches_loop_encoder_random():
    rng = np.random.default_rng(7)
    codes = rng.integers(0, 16, size=(37, 72), dtype=np.uint8)
    words = loop_pack_awq(codes.tolist())
    assert np.array_equal(orc.unpack_awq(words), codes)
    assert np.array_equal(wl.awq_pack_words(codes), words)


def test_unpack_of_random_words_round_trips():
    """Every uint32 is a legal word; decode then re-encode must give the word back bit for bit."""
    rng = np.random.default_rng(11)
    words = rng.integers(0, 2**32, size=(19, 13), dtype=np.uint64).astype(np.uint32)
    assert np.array_equal(loop_pack_awq(orc.unpack_awq(words).tolist()), words)


def test_bf16_bit_patterns():
    bits = np.array([0x3F80, 0xC000, 0x4300, 0x0000, 0x8000, 0x3DCD, 0x7F7F, 0x0001], dtype=np.uint16)
    want = [1.0, -2.0, 128.0, 0.0, -0.0, 0.10009765625, 3.3895313892515355e38, 2.0**-133]
    got = orc.bf16_bits_to_f64(bits)
    assert got.tolist() == want
    assert np.signbit(got[4]) and not np.signbit(got[3])
