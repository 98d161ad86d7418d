"""Pins of the oracle's 3-bit format (the W3A16, group-128 variant of Sec. 5 / App. "Quantization Detail").

The paper keeps its 3-bit checkpoint expanded to fp16 and prints no layout, so the layout is this library's own: every 32 codes
take three 32-bit words; code i < 30 of a block sits in word i // 10, five codes per half-word (bits 3j.. for j = i % 10 < 5,
bits 16 + 3(j - 5).. otherwise); bit b of code 30 is bit 15 of word b, bit b of code 31 is bit 31 of word b.  The pins use an
independent Python packer written from that sentence, a closed-form lossless group, the quantization rule in exact rational
arithmetic, brute-force argmin, and numpy's BLAS on independently unpacked weights.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2602_02711_b200 import inputs
from test_oracle_pins import reference_quantize_group, bf16_value


def python_pack3(codes_row):
    """32 codes -> three words, written from the documented layout (no code shared with the oracle)."""
    out = []
    for b in range(len(codes_row) // 32):
        w = [0, 0, 0]
        blk = [int(c) for c in codes_row[32 * b:32 * b + 32]]
        for i in range(30):
            j = i % 10
            shift = 3 * j if j < 5 else 16 + 3 * (j - 5)
            w[i // 10] |= blk[i] << shift
        for bit in range(3):
            w[bit] |= ((blk[30] >> bit) & 1) << 15
            w[bit] |= ((blk[31] >> bit) & 1) << 31
        out += w
    return out


def python_unpack3(words_row, K):
    codes = []
    for b in range(K // 32):
        w = [int(x) for x in words_row[3 * b:3 * b + 3]]
        for i in range(30):
            j = i % 10
            shift = 3 * j if j < 5 else 16 + 3 * (j - 5)
            codes.append((w[i // 10] >> shift) & 7)
        codes.append(sum(((w[bit] >> 15) & 1) << bit for bit in range(3)))
        codes.append(sum(((w[bit] >> 31) & 1) << bit for bit in range(3)))
    return codes


def test_pack_matches_the_documented_layout_and_round_trips():
    rng = np.random.default_rng(3)
    codes = rng.integers(0, 8, size=(5, 96), dtype=np.uint8)
    qw = oracle.pack(codes, 3)
    assert qw.shape == (5, 9)
    for n in range(5):
        assert list(qw[n]) == python_pack3(codes[n])
        assert python_unpack3(qw[n], 96) == list(codes[n])
    assert np.array_equal(oracle.unpack(qw, 96, 3), codes)


def test_every_code_value_at_every_position():
    for pos in range(32):
        for value in range(8):
            codes = np.zeros((1, 32), dtype=np.uint8)
            codes[0, pos] = value
            qw = oracle.pack(codes, 3)
            assert np.array_equal(oracle.unpack(qw, 32, 3), codes)
            # exactly the documented bits are set
            want = [0, 0, 0]
            if pos < 30:
                j = pos % 10
                want[pos // 10] = value << (3 * j if j < 5 else 16 + 3 * (j - 5))
            else:
                for bit in range(3):
                    want[bit] = ((value >> bit) & 1) << (15 if pos == 30 else 31)
            assert list(qw[0]) == want


def test_all_ones_block_fills_all_96_bits():
    qw = oracle.pack(np.full((1, 32), 7, dtype=np.uint8), 3)
    assert list(qw[0]) == [0xFFFFFFFF] * 3


def test_closed_form_ramp_is_lossless():
    # the eight levels (i - 4) / 64: lo = -4/64, hi = 3/64, s = (7/64) / 7 = 2^-6 exactly, zero = 4, code = i
    g = 128
    w = np.array([((i % 8) - 4) / 64.0 for i in range(g)])
    W = inputs.f64_to_bf16_bits(np.tile(w, (2, 2)))        # two rows, two groups each
    qw, sc, zp, codes = oracle.quantize(W, bits=3, group=g, return_codes=True)
    assert np.all(sc == 0x3C80)                            # 2^-6 as bf16
    assert np.all(zp == 4)
    assert np.array_equal(codes[0], np.tile(np.arange(g) % 8, 2))
    What, Wb = oracle.dequantize(qw, sc, zp, 2 * g, bits=3, group=g)
    assert np.array_equal(What, np.tile(w, (2, 2)))
    assert np.array_equal(Wb, W)


def test_quantize_matches_exact_rational_rule():
    N, K, g = 16, 256, 128
    W = inputs.weights(N, K, seed=31, index=3)
    qw, sc, zp, codes = oracle.quantize(W, bits=3, group=g, return_codes=True)
    assert codes.max() <= 7
    for n in range(N):
        for j in range(K // g):
            sb, z, q = reference_quantize_group(W[n, j * g:(j + 1) * g], 3)
            assert sc[n, j] == sb and zp[n, j] == z
            assert list(codes[n, j * g:(j + 1) * g]) == q
        assert python_unpack3(qw[n], K) == list(codes[n])


def test_codes_are_argmin_and_error_is_bounded():
    N, K, g = 4, 128, 128
    W = inputs.weights(N, K, seed=32)
    qw, sc, zp, codes = oracle.quantize(W, bits=3, group=g, return_codes=True)
    for n in range(N):
        s, z = bf16_value(int(sc[n, 0])), int(zp[n, 0])
        for k in range(K):
            w = bf16_value(int(W[n, k]))
            target = w / s + z
            best = min(range(8), key=lambda q: (abs(target - q), q % 2))
            assert abs(target - int(codes[n, k])) == abs(target - best)
            # inside the code range the error is at most half a step; the top code may clamp
            assert abs(w - s * (int(codes[n, k]) - z)) <= s * (Fraction(1, 2) + Fraction(7, 128))


def test_linear_matches_numpy_blas_on_independently_unpacked_weights():
    M, N, K, g = 5, 48, 512, 128
    W = inputs.weights(N, K, seed=33)
    X = inputs.activations(M, K, seed=33)
    qw, sc, zp = oracle.quantize(W, bits=3, group=g)
    codes = np.array([python_unpack3(qw[n], K) for n in range(N)], dtype=np.float64)
    s = inputs.bf16_bits_to_f64(sc).repeat(g, axis=1)
    z = zp.astype(np.float64).repeat(g, axis=1)
    What = s * (codes - z)
    Y = oracle.lowbit_linear(X, qw, sc, zp, bits=3, group=g)
    ref = inputs.bf16_bits_to_f64(X) @ What.T
    assert np.abs(Y - ref).max() <= 1e-12 * np.abs(ref).max()
    ms, ns = inputs.sample_outputs(M, N, 50, seed=1)
    got = oracle.sampled_linear(X, ms, ns, qweight=qw, scales=sc, zeros=zp, bits=3, group=g)
    assert np.array_equal(got, Y[ms, ns])
    # three bits lose more than four: the error against the bf16 layer is a few percent, not a few per mille
    dense = oracle.dense_linear(X, W)
    rel = np.abs(Y - dense).max() / np.abs(dense).max()
    assert 5e-3 < rel < 0.3


def test_bad_shapes_are_errors():
    with pytest.raises(oracle.OracleError):
        oracle.quantize(inputs.weights(2, 48, seed=1), bits=3, group=48)    # K not a multiple of 32
