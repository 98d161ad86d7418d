"""Parity of the 3-bit path (the W3A16, g = 128 variant of Sec. 5 / App. "Quantization Detail") with the CPU oracle.

Bars as for the 4-bit path: packed words, scales and zero points bit-exact; linear outputs within 2e-3 of the oracle on
the fp32 output, and within 5e-5 for the decode kernel, which multiplies exact integers (only the fp32 summation order
differs); the bf16 output is the nearest bf16 of the fp32 output; routed rows equal the unrouted call's rows bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_02711_b200 as dmr
from paper_2602_02711_b200 import inputs, QFormat, OUT_BF16, OUT_F32
from paper_2602_02711_b200.binding import OP_LOWBIT
from helpers import to_dev_bf16, bf16_to_bits, qweight_np, scales_np, zeros_np, rel_err

pytestmark = pytest.mark.gpu

TOL = 2e-3
TOL_EXACT_CODES = 5e-5


def quantize_both(W_bits, group):
    q = dmr.dmr_quantize(to_dev_bf16(W_bits), QFormat(3, group))
    ref = oracle.quantize(W_bits, bits=3, group=group)
    return q, ref


def assert_quant_equal(q, ref):
    qw, sc, zp = ref
    assert qweight_np(q).shape == qw.shape
    assert np.array_equal(qweight_np(q), qw)
    assert np.array_equal(scales_np(q), sc)
    assert np.array_equal(zeros_np(q), zp)


@pytest.mark.parametrize("N,K,group", [
    (512, 512, 128),     # the paper's group size
    (130, 640, 128),     # ragged N
    (37, 1024, 0),       # one group per row
    (24, 384, 96),       # groups of three blocks
    (5, 64, 32),         # one block per group
    (3, 32, 32),         # smallest legal sizes
])
def test_quantize_w3_bit_exact(N, K, group):
    W = inputs.weights(N, K, seed=0, index=3 * N + K)
    q, ref = quantize_both(W, group)
    assert_quant_equal(q, ref)


def test_quantize_w3_every_code_in_every_position():
    # row r, position k holds the value that quantizes to code (k + r) % 8: all eight codes pass through all 32
    # positions of a block, the two codes that are spread over bits 15 and 31 included
    N, K = 8, 128
    vals = np.array([[((k + r) % 8) / 8.0 for k in range(K)] for r in range(N)])
    W = inputs.f64_to_bf16_bits(vals)
    q, ref = quantize_both(W, 128)
    assert_quant_equal(q, ref)
    codes = oracle.unpack(qweight_np(q), K, 3)
    assert np.array_equal(codes, np.array([[(k + r) % 8 for k in range(K)] for r in range(N)], dtype=codes.dtype))


def test_quantize_w3_heavy_tails_and_ties():
    rng = np.random.default_rng(11)
    w = rng.standard_t(2, size=(96, 1024)) * 0.02
    W = inputs.f64_to_bf16_bits(np.clip(w, -1e3, 1e3))
    q, ref = quantize_both(W, 128)
    assert_quant_equal(q, ref)
    rows = np.zeros((3, 128))
    rows[0, :8] = [(2 * i + 1) / 16 for i in range(8)]   # exact ties between neighbouring codes (scale 1/8 after the 7/8 maximum)
    rows[0, 8] = 0.875
    rows[1, :] = -0.25
    rows[2, :] = np.linspace(-2.0e38, 2.0e38, 128)
    q, ref = quantize_both(inputs.f64_to_bf16_bits(rows), 128)
    assert_quant_equal(q, ref)


def test_quantize_w3_nonfinite_sets_status():
    W = inputs.weights(4, 256, seed=1)
    W[1, 77] = 0xFF80
    with pytest.raises(dmr.DmrError) as e:
        dmr.dmr_quantize(to_dev_bf16(W), QFormat(3, 128))
    assert e.value.code == 5


@pytest.mark.parametrize("group", [128, 32, 0])
def test_dequantize_w3_matches_oracle(group):
    N, K = 96, 512
    W = inputs.weights(N, K, seed=2, index=group)
    q, ref = quantize_both(W, group)
    What, Wb = oracle.dequantize(*ref, K, bits=3, group=group)
    got32 = dmr.dmr_dequantize(q, OUT_F32).cpu().numpy().astype(np.float64)
    assert np.array_equal(got32, What)
    assert np.array_equal(bf16_to_bits(dmr.dmr_dequantize(q, OUT_BF16)), Wb)


def run_case(M, N, K, group, seed=0, outlier=0.0):
    W = inputs.weights(N, K, seed=seed, index=N * 5 + K)
    X = inputs.activations(M, K, seed=seed, index=M, outlier_frac=outlier)
    q, ref = quantize_both(W, group)
    assert_quant_equal(q, ref)
    Xd = to_dev_bf16(X)
    Y32 = dmr.dmr_lowbit_linear(Xd, q, OUT_F32)
    Y16 = dmr.dmr_lowbit_linear(Xd, q, OUT_BF16)
    Yref = oracle.lowbit_linear(X, *ref, bits=3, group=group)
    y32 = Y32.cpu().numpy().astype(np.float64)
    assert rel_err(y32, Yref) <= TOL
    assert rel_err(y32, Yref) <= TOL_EXACT_CODES
    assert torch.equal(Y16, Y32.to(torch.bfloat16))
    return Y32


@pytest.mark.parametrize("M,N,K,group", [
    (1, 512, 512, 128),      # one token
    (8, 1024, 1024, 128),    # the 8-row instance, whole tiles (scale tables staged in shared memory)
    (5, 520, 640, 128),      # ragged N (tables read from global memory), K = 2.5 boxes: the last box is half used
    (16, 544, 896, 128),     # the 16-row instance, ragged N, odd number of chunks
    (13, 2048, 384, 128),    # fewer boxes than warps
    (16, 4736, 1792, 128),   # several tiles per CTA
    (4, 256, 1024, 256),     # groups of two chunks
    (3, 96, 768, 0),         # one group per row
    (29, 384, 512, 128),     # more rows than one launch takes: chunks of 16
])
def test_lowbit_linear_w3_decode(M, N, K, group):
    info = dmr.dmr_describe_dispatch(OP_LOWBIT, M, N, K, QFormat(3, group))
    assert info["kernel"] == "decode_w3"
    run_case(M, N, K, group)


@pytest.mark.parametrize("M,N,K,group", [
    (4, 100, 320, 64),       # groups of 64: not a multiple of the chunk
    (2, 64, 96, 32),
    (7, 33, 160, 160),
])
def test_lowbit_linear_w3_other_shapes(M, N, K, group):
    info = dmr.dmr_describe_dispatch(OP_LOWBIT, M, N, K, QFormat(3, group))
    assert info["kernel"] == "simple"
    run_case(M, N, K, group)


def test_lowbit_linear_w3_outlier_activations():
    run_case(8, 512, 2048, 128, seed=3, outlier=0.01)


def test_w3_row_independent_of_batch():
    # a row's result does not depend on the rows around it, within one instance of the kernel
    N, K = 1024, 1024
    W = inputs.weights(N, K, seed=4)
    X = inputs.activations(8, K, seed=4)
    q, _ = quantize_both(W, 128)
    Xd = to_dev_bf16(X)
    full = dmr.dmr_lowbit_linear(Xd, q, OUT_F32)
    for m in (0, 3, 7):
        one = dmr.dmr_lowbit_linear(Xd[m:m + 1].contiguous(), q, OUT_F32)
        assert torch.equal(one[0], full[m])


@pytest.mark.parametrize("M", [8, 16, 40])
def test_routed_linear_w3_rows_bitwise(M):
    N, K = 768, 1024
    W = inputs.weights(N, K, seed=6, index=M)
    X = inputs.activations(M, K, seed=6, index=M)
    mask = inputs.precision_mask(M, p_high=0.3, seed=6, index=M)
    q, ref = quantize_both(W, 128)
    Wd, Xd = to_dev_bf16(W), to_dev_bf16(X)
    md = torch.from_numpy(mask).cuda()
    Y = dmr.dmr_routed_linear(Xd, md, Wd, q, OUT_F32)
    Yl = dmr.dmr_lowbit_linear(Xd, q, OUT_F32)
    Yh = dmr.dmr_dense_linear(Xd, Wd, OUT_F32)
    for m in range(M):
        assert torch.equal(Y[m], Yh[m] if mask[m] else Yl[m])
    Yref = oracle.routed_linear(X, mask, W, *ref, bits=3, group=128)
    # 40 rows run on the tensor-core kernel, which rounds each dequantized weight once to fp16
    assert rel_err(Y.cpu().numpy().astype(np.float64), Yref) <= (TOL_EXACT_CODES if M <= 32 else 3e-4)


def test_w3_full_size_layer_sampled():
    # a whole decoder projection of the 7B configuration (3584 -> 18944), eight concurrent steps: sampled outputs
    N, K, M = 18944, 3584, 8
    W = inputs.weights(N, K, seed=7)
    X = inputs.activations(M, K, seed=7)
    q = dmr.dmr_quantize(to_dev_bf16(W), QFormat(3, 128))
    Y = dmr.dmr_lowbit_linear(to_dev_bf16(X), q, OUT_F32).cpu().numpy().astype(np.float64)
    ref = oracle.quantize(W, bits=3, group=128)
    assert_quant_equal(q, ref)
    ms, ns = inputs.sample_outputs(M, N, 4096, seed=7)
    want = oracle.sampled_linear(X, ms, ns, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=3, group=128)
    got = Y[ms, ns]
    assert float(np.abs(got - want).max() / np.abs(want).max()) <= TOL_EXACT_CODES
    assert np.isfinite(Y).all()


def test_w3_sizes_and_errors():
    assert dmr.lib().dmr_qweight_bytes(8, 128, QFormat(3, 128)) == 8 * 128 * 3 // 8
    assert dmr.lib().dmr_qweight_bytes(8, 100, QFormat(3, 0)) == 0          # K must be a multiple of 32
    W = to_dev_bf16(inputs.weights(4, 128, seed=0))
    with pytest.raises(dmr.DmrError):
        dmr.dmr_quantize(W, QFormat(3, 48))                          # groups hold whole blocks of 32 codes


TOL_PREFILL = 3e-4  # the tensor-core kernel rounds each dequantized weight once to fp16's 11 significant bits


@pytest.mark.parametrize("M,N,K,group", [
    (300, 640, 512, 128),     # three row tiles of 128 / 256, five feature tiles
    (150, 520, 1024, 128),    # ragged N and M
    (257, 256, 384, 64),      # groups of 64 = one stage, M just over a row tile
    (200, 128, 2048, 0),      # one group per row
])
def test_lowbit_linear_w3_prefill(M, N, K, group):
    info = dmr.dmr_describe_dispatch(OP_LOWBIT, M, N, K, QFormat(3, group))
    assert info["kernel"] == "prefill" and info["bits"] == 3
    W = inputs.weights(N, K, seed=11, index=N + K)
    X = inputs.activations(M, K, seed=11, index=M)
    q, ref = quantize_both(W, group)
    assert_quant_equal(q, ref)
    Xd = to_dev_bf16(X)
    Y32 = dmr.dmr_lowbit_linear(Xd, q, OUT_F32)
    Yref = oracle.lowbit_linear(X, *ref, bits=3, group=group)
    assert rel_err(Y32.cpu().numpy().astype(np.float64), Yref) <= TOL_PREFILL
    assert torch.equal(dmr.dmr_lowbit_linear(Xd, q, OUT_BF16), Y32.to(torch.bfloat16))


def test_w3_prefill_outliers_and_routed_rows():
    M, N, K = 200, 384, 1024
    W = inputs.weights(N, K, seed=12)
    X = inputs.activations(M, K, seed=12, outlier_frac=0.01)
    mask = inputs.precision_mask(M, p_high=0.3, seed=12)
    q, ref = quantize_both(W, 128)
    Wd, Xd = to_dev_bf16(W), to_dev_bf16(X)
    Yl = dmr.dmr_lowbit_linear(Xd, q, OUT_F32)
    assert rel_err(Yl.cpu().numpy().astype(np.float64), oracle.lowbit_linear(X, *ref, bits=3, group=128)) <= TOL_PREFILL
    Y = dmr.dmr_routed_linear(Xd, torch.from_numpy(mask).cuda(), Wd, q, OUT_F32)
    Yh = dmr.dmr_dense_linear(Xd, Wd, OUT_F32)
    for m in range(M):
        assert torch.equal(Y[m], Yh[m] if mask[m] else Yl[m])


def test_w3_prefill_7b_layer_sampled():
    N, K, M = 4096, 4096, 2048
    W = inputs.weights(N, K, seed=13)
    X = inputs.activations(M, K, seed=13)
    q = dmr.dmr_quantize(to_dev_bf16(W), QFormat(3, 128))
    ref = oracle.quantize(W, bits=3, group=128)
    assert_quant_equal(q, ref)
    Y = dmr.dmr_lowbit_linear(to_dev_bf16(X), q, OUT_F32).cpu().numpy().astype(np.float64)
    ms, ns = inputs.sample_outputs(M, N, 4096, seed=13)
    want = oracle.sampled_linear(X, ms, ns, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=3, group=128)
    assert float(np.abs(Y[ms, ns] - want).max() / np.abs(want).max()) <= TOL_PREFILL
    assert np.isfinite(Y).all()
