"""Pins for the CPU oracle: it is checked against things other than itself.

The paper prints no quantized value or layer output, so the pins are closed forms worked by
hand (tests/golden), exact rational arithmetic (fractions), brute force over all codes,
format invariants and numpy's float64 BLAS.  A plausible mistake in the oracle (dropped
zero point, wrong nibble order, transposed operand, rounding the wrong way, scale taken
before rounding to bf16) fails at least one of them.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2602_02711_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "closed_form_groups.txt")


# ---------- independent helpers (pure Python / numpy, no oracle code) ----------

def bf16_value(bits: int) -> Fraction:
    """Exact value of a finite bf16 bit pattern from its fields."""
    sign = -1 if bits & 0x8000 else 1
    e = (bits >> 7) & 0xFF
    m = bits & 0x7F
    if e == 0:
        return sign * Fraction(m, 1 << 7) * Fraction(2) ** (-126)
    return sign * (1 + Fraction(m, 1 << 7)) * Fraction(2) ** (e - 127)


def nearest_bf16_exact(x: Fraction) -> int:
    """Nearest positive bf16 pattern to a positive rational, ties to even, by exhaustive search."""
    assert x > 0
    best = None
    for bits in range(0x0001, 0x7F80):
        d = abs(bf16_value(bits) - x)
        if best is None or d < best[0] or (d == best[0] and bits % 2 == 0 and best[1] % 2 == 1):
            best = (d, bits)
    return best[1]


_BF16_TABLE = None


def nearest_bf16_fast(x: Fraction) -> int:
    """Same as nearest_bf16_exact, with a bisect over the sorted table of positive values."""
    global _BF16_TABLE
    if _BF16_TABLE is None:
        _BF16_TABLE = [bf16_value(b) for b in range(0, 0x7F80)]
    import bisect
    i = bisect.bisect_right(_BF16_TABLE, x) - 1  # table[i] <= x
    i = max(i, 0)
    if i + 1 >= len(_BF16_TABLE):
        return i
    dlo, dhi = x - _BF16_TABLE[i], _BF16_TABLE[i + 1] - x
    if dlo < dhi:
        return i
    if dhi < dlo:
        return i + 1
    return i if i % 2 == 0 else i + 1


def round_half_even(x: Fraction) -> int:
    f = x.numerator // x.denominator  # floor
    r = x - f
    if r < Fraction(1, 2):
        return f
    if r > Fraction(1, 2):
        return f + 1
    return f if f % 2 == 0 else f + 1


def reference_quantize_group(wbits, bits):
    """The quantization rule in exact rational arithmetic."""
    qmax = (1 << bits) - 1
    w = [bf16_value(int(b)) for b in wbits]
    lo = min(Fraction(0), min(w))
    hi = max(Fraction(0), max(w))
    if hi == lo:
        sb = 0x3F80
    else:
        sb = nearest_bf16_fast((hi - lo) / qmax)
        sb = max(sb, 0x0080)
    s = bf16_value(sb)
    z = min(max(round_half_even(-lo / s), 0), qmax)
    q = [min(max(round_half_even(x / s) + z, 0), qmax) for x in w]
    return sb, z, q


def python_pack(codes_row, bits):
    per = 32 // bits
    out = []
    for j in range(len(codes_row) // per):
        w = 0
        for i in range(per):
            w |= int(codes_row[j * per + i]) << (bits * i)
        out.append(w)
    return out


# ---------- bf16 conversion ----------

def test_bf16_widen_matches_fields():
    for bits in [0x0000, 0x0080, 0x3F80, 0x3C80, 0xBF80, 0x4049, 0x7F7F, 0x0001, 0x8001, 0x3DCD]:
        assert Fraction(oracle.bf16_to_f64(bits)) == bf16_value(bits)


def test_bf16_rne_against_exhaustive_search():
    rng = np.random.default_rng(1)
    xs = list(np.exp(rng.uniform(-20, 20, size=40)))
    # exact ties between neighbours: must go to the even pattern
    for b in [0x3F80, 0x3F81, 0x3C7F, 0x4000, 0x00FF]:
        xs.append(float((bf16_value(b) + bf16_value(b + 1)) / 2))
    for x in xs:
        assert oracle.f64_to_bf16_rne(x) == nearest_bf16_exact(Fraction(x))
        assert oracle.f64_to_bf16_rne(-x) == (0x8000 | nearest_bf16_exact(Fraction(x)))
    assert oracle.f64_to_bf16_rne(0.0) == 0


def test_bf16_rne_against_second_implementation():
    rng = np.random.default_rng(2)
    x = rng.standard_normal(20000) * np.exp(rng.uniform(-8, 8, size=20000))
    want = inputs.f64_to_bf16_bits(x)
    got = np.array([oracle.f64_to_bf16_rne(v) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)


def test_bf16_rne_no_double_rounding():
    # value just above a bf16 tie: rounding through float32 first would land on the tie and go to even
    x = float.fromhex("0x1.010000000001p+0")
    assert oracle.f64_to_bf16_rne(x) == 0x3F81
    x = float.fromhex("0x1.00ffffffffffp+0")
    assert oracle.f64_to_bf16_rne(x) == 0x3F80


# ---------- pack / unpack ----------

@pytest.mark.parametrize("bits", [4, 8])
def test_pack_unpack_bijection(bits):
    rng = np.random.default_rng(3)
    codes = rng.integers(0, 1 << bits, size=(7, 256), dtype=np.uint8)
    qw = oracle.pack(codes, bits)
    assert qw.shape == (7, 256 * bits // 32)
    assert np.array_equal(oracle.unpack(qw, 256, bits), codes)
    for n in range(7):
        assert list(qw[n]) == python_pack(codes[n], bits)


@pytest.mark.parametrize("bits", [4, 8])
def test_pack_one_hot_sets_documented_bits(bits):
    per = 32 // bits
    K = 2 * per
    for k in range(K):
        for code in range(1 << bits):
            codes = np.zeros((1, K), dtype=np.uint8)
            codes[0, k] = code
            qw = oracle.pack(codes, bits)
            want = [0, 0]
            want[k // per] = code << (bits * (k % per))
            assert list(qw[0]) == want


def test_nibble_order_is_little_endian():
    codes = np.arange(8, dtype=np.uint8).reshape(1, 8)
    assert oracle.pack(codes, 4)[0, 0] == 0x76543210
    codes = np.array([[1, 2, 3, 4]], dtype=np.uint8)
    assert oracle.pack(codes, 8)[0, 0] == 0x04030201


# ---------- quantization ----------

def _golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, bits, wexpr, count, sb, zero, qexpr = [c.strip() for c in line.split("|")]
            rows.append((name, int(bits), wexpr, int(count), int(sb, 16), int(zero), qexpr))
    return rows


@pytest.mark.parametrize("row", _golden_rows(), ids=lambda r: r[0])
def test_closed_form_groups(row):
    name, bits, wexpr, count, sb, zero, qexpr = row
    w = np.array([eval(wexpr, {"i": i}) for i in range(count)], dtype=np.float64)
    wb = inputs.f64_to_bf16_bits(w)
    assert np.array_equal(inputs.bf16_bits_to_f64(wb), w), "fixture weights must be exact in bf16"
    per = 32 // bits
    reps = 1
    while (count * reps) % per or (count * reps) % 32:
        reps += 1
    W = np.tile(wb, reps).reshape(1, -1)
    K = W.shape[1]
    qw, sc, zp, codes = oracle.quantize(W, bits=bits, group=count, return_codes=True)
    assert (sc == sb).all()
    assert (zp == zero).all()
    want = np.array([eval(qexpr, {"i": i}) for i in range(count)], dtype=np.uint8)
    assert np.array_equal(codes[0], np.tile(want, reps))
    What, Wb = oracle.dequantize(qw, sc, zp, K, bits=bits, group=count)
    if name.startswith("ramp") or name.endswith("ramp4"):
        # lossless cases: dequantized weights equal the inputs bit for bit
        assert np.array_equal(What[0], np.tile(w, reps))
        assert np.array_equal(Wb[0], np.tile(wb, reps))


@pytest.mark.parametrize("bits,group", [(4, 128), (4, 64), (8, 128)])
def test_quantize_matches_exact_rational_rule(bits, group):
    N, K = 24, 2 * group
    W = inputs.weights(N, K, seed=11, index=bits + group)
    qw, sc, zp, codes = oracle.quantize(W, bits=bits, group=group, return_codes=True)
    for n in range(N):
        for j in range(K // group):
            sb, z, q = reference_quantize_group(W[n, j * group:(j + 1) * group], bits)
            assert sc[n, j] == sb
            assert zp[n, j] == z
            assert list(codes[n, j * group:(j + 1) * group]) == q
    assert np.array_equal(oracle.unpack(qw, K, bits), codes)


def test_quantize_per_channel_int8_matches_rule():
    N, K = 6, 512
    W = inputs.weights(N, K, seed=12)
    qw, sc, zp, codes = oracle.quantize(W, bits=8, group=0, return_codes=True)
    assert sc.shape == (N, 1) and zp.shape == (N, 1)
    for n in range(N):
        sb, z, q = reference_quantize_group(W[n], 8)
        assert sc[n, 0] == sb and zp[n, 0] == z and list(codes[n]) == q


def test_ties_round_half_to_even():
    # s = 2^-6 exactly (range -8/64 .. 7/64); weights at odd multiples of 2^-7 are exact ties
    base = [(i - 8) / 64 for i in range(16)]
    ties = [1 / 128, 3 / 128, 5 / 128, -1 / 128, -3 / 128, 11 / 128]
    w = np.array(base + ties + [0.0] * (32 - 22), dtype=np.float64)
    W = inputs.f64_to_bf16_bits(w).reshape(1, 32)
    _, sc, zp, codes = oracle.quantize(W, bits=4, group=32, return_codes=True)
    assert sc[0, 0] == 0x3C80 and zp[0, 0] == 8
    # 0.5 -> 0, 1.5 -> 2, 2.5 -> 2, -0.5 -> 0, -1.5 -> -2, 5.5 -> 6   (then + z)
    assert list(codes[0, 16:22]) == [8, 10, 10, 8, 6, 14]


@pytest.mark.parametrize("bits,group", [(4, 128), (4, 64), (8, 0)])
def test_grid_zero_and_error_bound_invariants(bits, group):
    N, K = 16, 512
    qmax = (1 << bits) - 1
    W = inputs.weights(N, K, seed=13, index=bits)
    # plant exact zeros
    W[:, ::17] = 0
    g = K if group == 0 else group
    qw, sc, zp, codes = oracle.quantize(W, bits=bits, group=group, return_codes=True)
    What, _ = oracle.dequantize(qw, sc, zp, K, bits=bits, group=group)
    w = inputs.bf16_bits_to_f64(W)
    s = np.repeat(inputs.bf16_bits_to_f64(sc), g, axis=1)
    z = np.repeat(zp.astype(np.float64), g, axis=1)
    ratio = What / s
    assert np.array_equal(ratio, np.rint(ratio))                      # on the grid
    assert (ratio >= -z).all() and (ratio <= qmax - z).all()          # inside the code range
    assert (What[w == 0] == 0).all()                                  # zero is exact
    assert (codes[w == 0] == zp.repeat(g, axis=1)[w == 0]).all()
    err = np.abs(w - What)
    assert (err <= s * (0.5 + qmax * 2.0 ** -7)).all()
    unclamped = (codes > 0) & (codes < qmax)
    assert (err[unclamped] <= s[unclamped] / 2).all()
    # the group minimum maps to code 0 whenever it is negative
    for n in range(N):
        for j in range(K // g):
            seg = w[n, j * g:(j + 1) * g]
            k = int(np.argmin(seg))
            if seg[k] < 0:
                assert codes[n, j * g + k] == 0


def test_codes_are_argmin_by_brute_force():
    N, K, bits, group = 4, 64, 4, 64
    W = inputs.weights(N, K, seed=14)
    _, sc, zp, codes = oracle.quantize(W, bits=bits, group=group, return_codes=True)
    for n in range(N):
        s = bf16_value(int(sc[n, 0]))
        z = int(zp[n, 0])
        for k in range(K):
            t = bf16_value(int(W[n, k])) / s + z
            dist = [abs(t - q) for q in range(16)]
            best = min(dist)
            winners = [q for q in range(16) if dist[q] == best]
            q = int(codes[n, k])
            assert q in winners
            if len(winners) == 2:
                # tie: rint picks the even value of w/s, i.e. q - z even
                assert (q - z) % 2 == 0


def test_special_groups():
    g = 128
    rows = np.zeros((4, g), dtype=np.float64)
    rows[1, :] = 0.03125
    rows[2, :] = -0.03125
    rows[3, 5] = 2.0 ** -130  # subnormal-range weight: scale guard keeps s >= 2^-126
    # bf16 has subnormals; build that row's bits by hand
    W = np.zeros((4, g), dtype=np.uint16)
    W[:3] = inputs.f64_to_bf16_bits(rows[:3])
    W[3, 5] = 0x0008  # 8 * 2^-133 = 2^-130
    _, sc, zp, codes = oracle.quantize(W, bits=4, group=g, return_codes=True)
    assert sc[0, 0] == 0x3F80 and zp[0, 0] == 0 and (codes[0] == 0).all()
    assert zp[1, 0] == 0 and (codes[1] == 15).all()
    assert zp[2, 0] == 15 and (codes[2] == 0).all()
    assert sc[3, 0] == 0x0080 and zp[3, 0] == 0 and codes[3, 5] == 0


def test_nonfinite_weight_is_an_error():
    W = inputs.weights(2, 128, seed=15)
    W[1, 7] = 0x7F80
    with pytest.raises(oracle.OracleError) as e:
        oracle.quantize(W, bits=4, group=128)
    assert e.value.code == oracle.ERR_NONFINITE
    W[1, 7] = 0x7FC1
    with pytest.raises(oracle.OracleError):
        oracle.quantize(W, bits=4, group=128)


def test_bad_shapes_are_errors():
    W = inputs.weights(2, 96, seed=16)
    with pytest.raises(oracle.OracleError):
        oracle.quantize(W, bits=4, group=64)


def test_dequantize_formula_and_rounding():
    N, K = 8, 256
    W = inputs.weights(N, K, seed=17)
    qw, sc, zp, codes = oracle.quantize(W, bits=4, group=128, return_codes=True)
    What, Wb = oracle.dequantize(qw, sc, zp, K, bits=4, group=128)
    for n in range(N):
        for k in range(0, K, 37):
            exact = bf16_value(int(sc[n, k // 128])) * (int(codes[n, k]) - int(zp[n, k // 128]))
            assert Fraction(What[n, k]) == exact
            if exact != 0:
                want = nearest_bf16_fast(abs(exact)) | (0x8000 if exact < 0 else 0)
                assert Wb[n, k] == want


# ---------- linear layers ----------

@pytest.mark.parametrize("bits,group", [(4, 128), (8, 0)])
def test_lowbit_linear_matches_numpy_blas(bits, group):
    M, N, K = 5, 48, 512
    W = inputs.weights(N, K, seed=20)
    X = inputs.activations(M, K, seed=20)
    qw, sc, zp = oracle.quantize(W, bits=bits, group=group)
    What, Wb = oracle.dequantize(qw, sc, zp, K, bits=bits, group=group)
    Y = oracle.lowbit_linear(X, qw, sc, zp, bits=bits, group=group)
    ref = inputs.bf16_bits_to_f64(X) @ What.T
    assert Y.shape == (M, N)
    assert np.abs(Y - ref).max() <= 1e-12 * np.abs(ref).max()
    Yb = oracle.lowbit_linear(X, qw, sc, zp, bits=bits, group=group, rounded=True)
    refb = inputs.bf16_bits_to_f64(X) @ inputs.bf16_bits_to_f64(Wb).T
    assert np.abs(Yb - refb).max() <= 1e-12 * np.abs(refb).max()
    assert np.abs(Yb - Y).max() > 0  # the two differ (rounded weights), but only slightly
    assert np.abs(Yb - Y).max() <= 2e-3 * np.abs(Y).max()


def test_dense_linear_matches_numpy_blas_and_is_not_transposed():
    M, N, K = 3, 40, 256
    W = inputs.weights(N, K, seed=21)
    X = inputs.activations(M, K, seed=21)
    Y = oracle.dense_linear(X, W)
    ref = inputs.bf16_bits_to_f64(X) @ inputs.bf16_bits_to_f64(W).T
    assert np.abs(Y - ref).max() <= 1e-12 * np.abs(ref).max()


def test_identity_and_one_hot_activations_pick_weights():
    N, K = 16, 128
    W = inputs.weights(N, K, seed=22)
    qw, sc, zp = oracle.quantize(W, bits=4, group=128)
    What, _ = oracle.dequantize(qw, sc, zp, K, bits=4, group=128)
    eye = inputs.f64_to_bf16_bits(np.eye(K))
    assert np.array_equal(oracle.lowbit_linear(eye, qw, sc, zp, bits=4, group=128), What.T)
    assert np.array_equal(oracle.dense_linear(eye, W), inputs.bf16_bits_to_f64(W).T)
    onehot = np.zeros((1, K))
    onehot[0, 77] = 2.0
    Y = oracle.lowbit_linear(inputs.f64_to_bf16_bits(onehot), qw, sc, zp, bits=4, group=128)
    assert np.array_equal(Y[0], 2.0 * What[:, 77])


def test_lossless_layer_lowbit_equals_dense():
    # every group is the 16-value ramp: quantization is lossless, so both layers agree exactly
    N, K = 8, 256
    ramp = np.array([((i % 16) - 8) / 64 for i in range(K)])
    rng = np.random.default_rng(23)
    Wf = np.stack([np.roll(ramp, int(rng.integers(0, 16))) for _ in range(N)])
    W = inputs.f64_to_bf16_bits(Wf)
    X = inputs.activations(4, K, seed=23)
    qw, sc, zp = oracle.quantize(W, bits=4, group=128)
    assert np.array_equal(oracle.lowbit_linear(X, qw, sc, zp), oracle.dense_linear(X, W))


def test_routed_rows_and_permutation():
    M, N, K = 12, 24, 256
    W = inputs.weights(N, K, seed=24)
    X = inputs.activations(M, K, seed=24)
    mask = inputs.precision_mask(M, 0.4, seed=24)
    assert 0 < mask.sum() < M
    qw, sc, zp = oracle.quantize(W, bits=4, group=128)
    Y = oracle.routed_linear(X, mask, W, qw, sc, zp)
    Yl = oracle.lowbit_linear(X, qw, sc, zp)
    Yh = oracle.dense_linear(X, W)
    for m in range(M):
        assert np.array_equal(Y[m], Yh[m] if mask[m] else Yl[m])
    assert np.array_equal(oracle.routed_linear(X, np.zeros(M, np.uint8), W, qw, sc, zp), Yl)
    assert np.array_equal(oracle.routed_linear(X, np.ones(M, np.uint8), W, qw, sc, zp), Yh)
    perm = np.random.default_rng(24).permutation(M)
    Yp = oracle.routed_linear(X[perm], mask[perm], W, qw, sc, zp)
    assert np.array_equal(Yp, Y[perm])
    # any non-zero mask byte means high precision
    mask2 = mask * 7
    assert np.array_equal(oracle.routed_linear(X, mask2, W, qw, sc, zp), Y)


def test_route_partition_is_stable():
    mask = inputs.precision_mask(64, 0.3, seed=25)
    ih, il = oracle.route_partition(mask)
    assert list(ih) == [m for m in range(64) if mask[m]]
    assert list(il) == [m for m in range(64) if not mask[m]]
    ih, il = oracle.route_partition(np.zeros(5, np.uint8))
    assert len(ih) == 0 and list(il) == [0, 1, 2, 3, 4]


def test_sampled_outputs_equal_full_outputs():
    M, N, K = 6, 32, 256
    W = inputs.weights(N, K, seed=26)
    X = inputs.activations(M, K, seed=26)
    mask = inputs.precision_mask(M, 0.5, seed=26)
    qw, sc, zp = oracle.quantize(W, bits=4, group=128)
    ms, ns = inputs.sample_outputs(M, N, 20, seed=26)
    Y = oracle.routed_linear(X, mask, W, qw, sc, zp)
    got = oracle.sampled_linear(X, ms, ns, mask=mask, W=W, qweight=qw, scales=sc, zeros=zp)
    assert np.array_equal(got, Y[ms, ns])
    got = oracle.sampled_linear(X, ms, ns, qweight=qw, scales=sc, zeros=zp)
    assert np.array_equal(got, oracle.lowbit_linear(X, qw, sc, zp)[ms, ns])
    got = oracle.sampled_linear(X, ms, ns, W=W)
    assert np.array_equal(got, oracle.dense_linear(X, W)[ms, ns])


def test_config1_quantization_error_is_small():
    # K=512, N=512, INT4 g=128: the first parity configuration; the oracle finishes in seconds
    W = inputs.weights(512, 512, seed=0)
    X = inputs.activations(4, 512, seed=0)
    qw, sc, zp = oracle.quantize(W, bits=4, group=128)
    Yl = oracle.lowbit_linear(X, qw, sc, zp)
    Yh = oracle.dense_linear(X, W)
    rel = np.abs(Yl - Yh).max() / np.abs(Yh).max()
    assert 0 < rel < 0.25  # 4-bit noise is visible but bounded
