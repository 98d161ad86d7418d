"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Bars: packed weights, scales and zeros bit-exact; linear outputs max|Y - Y_ref| / max|Y_ref|
<= 2e-3 on the fp32 output (fp32 accumulation); the bf16 output is the nearest bf16 of the fp32
output of the same kernel; routed rows equal the unrouted call's rows bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_02711_b200 as dmr
from paper_2602_02711_b200 import inputs, QFormat, OUT_BF16, OUT_F32
from helpers import (to_dev_bf16, bf16_to_bits, qweight_np, scales_np, zeros_np, rel_err)

pytestmark = pytest.mark.gpu

TOL = 2e-3          # acceptance bound on the fp32 output
TOL_PREFILL = 3e-4  # fp16 rounding of the dequantized weights: ~2^-12 per weight, ~1e-4 rms on the outputs
TOL_ROUNDED = 5e-5  # against the oracle run with the nearest-bf16 dequantized weights: only fp32
                    # summation order differs (bound ~ K * 2^-24 * sum|x||w| / max|Y|)


def quantize_both(W_bits, bits, group):
    q = dmr.dmr_quantize(to_dev_bf16(W_bits), QFormat(bits, group))
    ref = oracle.quantize(W_bits, bits=bits, group=group)
    return q, ref


def assert_quant_equal(q, ref):
    qw, sc, zp = ref
    assert np.array_equal(qweight_np(q), qw)
    assert np.array_equal(scales_np(q), sc)
    assert np.array_equal(zeros_np(q), zp)


# ---------------- quantize / dequantize ----------------

@pytest.mark.parametrize("N,K,bits,group", [
    (512, 512, 4, 128),      # first parity configuration
    (520, 640, 4, 64),       # ragged N, g = 64
    (37, 1024, 8, 0),        # INT8 per-channel
    (64, 256, 8, 128),
    (16, 2048, 4, 0),        # INT4 per-channel
    (3, 32, 4, 32),          # smallest legal sizes
])
def test_quantize_bit_exact(N, K, bits, group):
    W = inputs.weights(N, K, seed=0, index=N + K)
    q, ref = quantize_both(W, bits, group)
    assert_quant_equal(q, ref)


def test_quantize_special_groups_and_ties():
    g = 128
    rows = np.zeros((6, g), dtype=np.float64)
    rows[1, :] = 0.03125
    rows[2, :] = -0.03125
    rows[3, :16] = [(i - 8) / 64 for i in range(16)]
    rows[3, 16:22] = [1 / 128, 3 / 128, 5 / 128, -1 / 128, -3 / 128, 11 / 128]   # exact ties
    rows[4, :] = np.linspace(-3.0e38, 3.0e38, g)                                  # near the bf16 limits
    W = inputs.f64_to_bf16_bits(rows)
    W[5, 5] = 0x0008   # subnormal weight: the scale guard applies
    W[5, 6] = 0x8003
    q, ref = quantize_both(W, 4, g)
    assert_quant_equal(q, ref)
    q, ref = quantize_both(W, 8, 0)
    assert_quant_equal(q, ref)


def test_quantize_heavy_tailed_weights_bit_exact():
    # wide dynamic range inside groups: many codes sit on rounding boundaries
    rng = np.random.default_rng(5)
    w = rng.standard_t(2, size=(128, 1024)) * 0.02
    W = inputs.f64_to_bf16_bits(np.clip(w, -1e3, 1e3))
    for bits, group in [(4, 128), (4, 64), (8, 0)]:
        q, ref = quantize_both(W, bits, group)
        assert_quant_equal(q, ref)


def test_quantize_nonfinite_sets_status():
    W = inputs.weights(4, 256, seed=1)
    W[2, 100] = 0x7F80
    with pytest.raises(dmr.DmrError) as e:
        dmr.dmr_quantize(to_dev_bf16(W), QFormat(4, 128))
    assert e.value.code == 5
    with pytest.raises(oracle.OracleError):
        oracle.quantize(W, bits=4, group=128)


@pytest.mark.parametrize("bits,group", [(4, 128), (4, 64), (8, 0)])
def test_dequantize_matches_oracle(bits, group):
    N, K = 96, 512
    W = inputs.weights(N, K, seed=2, index=bits)
    q, ref = quantize_both(W, bits, group)
    What, Wb = oracle.dequantize(*ref, K, bits=bits, group=group)
    got32 = dmr.dmr_dequantize(q, OUT_F32).cpu().numpy().astype(np.float64)
    assert np.array_equal(got32, What)           # s*(q-z) is exact in fp32
    got16 = bf16_to_bits(dmr.dmr_dequantize(q, OUT_BF16))
    assert np.array_equal(got16, Wb)


# ---------------- linear layers ----------------

def run_lowbit_case(M, N, K, bits, group, seed=0, outlier=0.0):
    W = inputs.weights(N, K, seed=seed, index=N * 7 + K)
    X = inputs.activations(M, K, seed=seed, index=M, outlier_frac=outlier)
    q, ref = quantize_both(W, bits, group)
    assert_quant_equal(q, ref)
    Xd = to_dev_bf16(X)
    Y32 = dmr.dmr_lowbit_linear(Xd, q, OUT_F32)
    Y16 = dmr.dmr_lowbit_linear(Xd, q, OUT_BF16)
    Yref = oracle.lowbit_linear(X, *ref, bits=bits, group=group)
    y32 = Y32.cpu().numpy().astype(np.float64)
    assert rel_err(y32, Yref) <= TOL
    # sharper check: the decode kernels and the split-K tensor-core kernel multiply exact integers
    # (only fp32 summation order differs from the oracle); the persistent prefill kernel (M > 32)
    # rounds each dequantized weight once to fp16's 11 significant bits
    assert rel_err(y32, Yref) <= (TOL_ROUNDED if M <= 32 else TOL_PREFILL)
    # bf16 output = nearest bf16 of the same accumulators
    assert torch.equal(Y16, Y32.to(torch.bfloat16))
    # determinism
    assert torch.equal(dmr.dmr_lowbit_linear(Xd, q, OUT_F32), Y32)
    return rel_err(y32, Yref)


@pytest.mark.parametrize("M", [1, 4])
def test_config1_lowbit_linear(M):
    run_lowbit_case(M, 512, 512, 4, 128)


@pytest.mark.parametrize("M,N,K,bits,group", [
    (8, 520, 640, 4, 128),     # ragged N (not a multiple of 16), several k-steps per warp
    (16, 1000, 1024, 4, 128),
    (13, 2072, 2048, 4, 64),   # g = 64, M between the 8- and 16-row tiles
    (5, 264, 4096, 4, 0),      # per-channel INT4
    (3, 200, 1024, 8, 0),      # INT8 per-channel
    (16, 328, 512, 8, 128),
    (1, 24, 128, 4, 128),      # smallest K the decode kernel takes
    (2, 40, 160, 4, 32),       # K not a multiple of 128: any-shape kernel
    (24, 1000, 1024, 4, 128),  # 17 .. 32 rows: two chunks of the 16-row instance of the 4-bit decode kernel
    (32, 520, 2048, 8, 0),     # 8-bit: the 32-row instance of the streaming kernel
    (17, 4096, 4096, 4, 64),   # g = 64, one full and one one-row chunk
    (31, 22016, 512, 4, 128),  # many tiles per CTA, two boxes per row
    (40, 300, 512, 4, 128),    # M above the decode limit: tensor-core GEMM, ragged N and M
    (33, 136, 384, 8, 0),
    (64, 256, 4096, 4, 128),   # few tiles, long K: split-K with ordered reduction
    (64, 250, 4096, 4, 128),   # ... and N not a multiple of 4: the sums of the splits go one feature per thread
    (130, 264, 1024, 4, 64),   # two column blocks, g = 64
    (100, 200, 2048, 8, 0),    # INT8 per-channel: one group spans all of K
    (300, 520, 640, 4, 128),
    (257, 128, 256, 4, 0),
])
def test_lowbit_linear_shapes(M, N, K, bits, group):
    run_lowbit_case(M, N, K, bits, group, seed=3)


@pytest.mark.parametrize("M,N,K,bits,group", [
    (8, 22016, 2048, 4, 128),  # 688 tiles of 32 rows, 8 boxes per row: half of the warps have no box
    (3, 4224, 768, 4, 128),    # 3 boxes per row: most warps idle, sums of three warps
    (7, 1000, 4096, 8, 128),   # INT8, ragged N: streaming kernel in cluster mode (8 feature groups, 8 clusters)
    (1, 4096, 4096, 4, 64),    # g = 64 (64-wide chunks, four per box)
    (8, 136, 11008, 4, 0),     # per-channel scales (tables not staged as pairs), 43 boxes per row: uneven shares (2 and 3 boxes)
])
def test_lowbit_linear_cluster_mode_shapes(M, N, K, bits, group):
    """Layers with up to 8 rows whose k range divides unevenly among the warps of a CTA (4-bit decode kernel)
    or among the CTAs of a thread-block cluster (8-bit streaming kernel)."""
    run_lowbit_case(M, N, K, bits, group, seed=5)


def test_prefill_accuracy_margin_and_extreme_ranges():
    # the prefill kernel multiplies fp16 operands after rescaling activation rows and weight scales by
    # powers of two: the error against the exact oracle stays well inside the 2e-3 bound ...
    assert run_lowbit_case(300, 520, 640, 4, 128, seed=16) <= 4e-4
    assert run_lowbit_case(200, 264, 1024, 8, 0, seed=17) <= 4e-4
    # ... and rows or layers far outside fp16's own range lose nothing (per row: the rows differ by 2^120)
    M, N, K = 160, 264, 512
    Wf = inputs.bf16_bits_to_f64(inputs.weights(N, K, seed=18)) * 2.0 ** -40
    W = inputs.f64_to_bf16_bits(Wf)
    Xf = inputs.bf16_bits_to_f64(inputs.activations(M, K, seed=18))
    Xf[0] *= 2.0 ** 60
    Xf[1] *= 2.0 ** -60
    X = inputs.f64_to_bf16_bits(Xf)
    q, ref = quantize_both(W, 4, 128)
    assert_quant_equal(q, ref)
    Y = dmr.dmr_lowbit_linear(to_dev_bf16(X), q, OUT_F32).cpu().numpy().astype(np.float64)
    Yref = oracle.lowbit_linear(X, *ref, bits=4, group=128)
    assert np.isfinite(Y).all()
    for m in (0, 1, 2, M - 1):
        assert np.abs(Y[m] - Yref[m]).max() / np.abs(Yref[m]).max() <= 1e-3


def test_lowbit_linear_with_outlier_channels():
    run_lowbit_case(8, 512, 5120, 4, 64, seed=4, outlier=0.01)


@pytest.mark.parametrize("M,N,K", [(1, 512, 512), (4, 512, 512), (16, 1000, 1024), (11, 72, 4096), (27, 1000, 2048),
                                   (3, 40, 200), (40, 300, 512), (64, 256, 4096), (200, 264, 1024),
                                   (300, 520, 640), (1000, 130, 192)])
def test_dense_linear(M, N, K):
    W = inputs.weights(N, K, seed=6, index=N)
    X = inputs.activations(M, K, seed=6, index=M)
    Xd, Wd = to_dev_bf16(X), to_dev_bf16(W)
    Y32 = dmr.dmr_dense_linear(Xd, Wd, OUT_F32)
    Y16 = dmr.dmr_dense_linear(Xd, Wd, OUT_BF16)
    Yref = oracle.dense_linear(X, W)
    assert rel_err(Y32.cpu().numpy().astype(np.float64), Yref) <= TOL_ROUNDED
    assert torch.equal(Y16, Y32.to(torch.bfloat16))
    assert torch.equal(dmr.dmr_dense_linear(Xd, Wd, OUT_F32), Y32)


def test_lossless_layer_lowbit_equals_dense_kernel():
    # every group is the 16-value ramp, so dequantized weights equal the bf16 weights exactly
    N, K = 256, 1024
    ramp = np.array([((i % 16) - 8) / 64 for i in range(K)])
    rng = np.random.default_rng(7)
    Wf = np.stack([np.roll(ramp, int(rng.integers(0, 16))) for _ in range(N)])
    W = inputs.f64_to_bf16_bits(Wf)
    X = inputs.activations(8, K, seed=7)
    q, ref = quantize_both(W, 4, 128)
    assert_quant_equal(q, ref)
    Yl = dmr.dmr_lowbit_linear(to_dev_bf16(X), q, OUT_F32).cpu().numpy().astype(np.float64)
    Yd = dmr.dmr_dense_linear(to_dev_bf16(X), to_dev_bf16(W), OUT_F32).cpu().numpy().astype(np.float64)
    Yref = oracle.dense_linear(X, W)
    assert rel_err(Yl, Yref) <= TOL_ROUNDED and rel_err(Yd, Yref) <= TOL_ROUNDED


def test_one_hot_activations_pick_single_weights():
    N, K = 64, 512
    W = inputs.weights(N, K, seed=8)
    q, ref = quantize_both(W, 4, 128)
    What, _ = oracle.dequantize(*ref, K, bits=4, group=128)
    Xf = np.zeros((8, K))
    cols = [0, 1, 5, 127, 128, 300, 510, 511]
    for m, c in enumerate(cols):
        Xf[m, c] = 1.0
    Y = dmr.dmr_lowbit_linear(to_dev_bf16(inputs.f64_to_bf16_bits(Xf)), q, OUT_F32).cpu().numpy()
    # the kernel multiplies exact integers q - zero and scales the group sum in fp32: no rounding at all
    assert np.array_equal(Y.astype(np.float64), What[:, cols].T)


# ---------------- routing ----------------

@pytest.mark.parametrize("M", [0, 1, 5, 64, 1000, 1024, 3000])
def test_route_partition(M):
    mask = inputs.precision_mask(max(M, 1), 0.3, seed=9, index=M)[:M]
    md = torch.from_numpy(mask).cuda() if M else torch.zeros(0, dtype=torch.uint8, device="cuda")
    ih, il, counts = dmr.dmr_route_partition(md)
    want_h, want_l = oracle.route_partition(mask) if M else (np.zeros(0, np.int32), np.zeros(0, np.int32))
    c = counts.cpu().numpy()
    assert c[0] == len(want_h) and c[1] == len(want_l)
    assert np.array_equal(ih.cpu().numpy()[:c[0]], want_h)
    assert np.array_equal(il.cpu().numpy()[:c[1]], want_l)


def routed_case(M, N, K, bits, group, mask, seed=10):
    W = inputs.weights(N, K, seed=seed, index=N)
    X = inputs.activations(M, K, seed=seed, index=M)
    q, ref = quantize_both(W, bits, group)
    Xd, Wd = to_dev_bf16(X), to_dev_bf16(W)
    md = torch.from_numpy(mask).cuda()
    for out in (OUT_F32, OUT_BF16):
        sentinel = torch.full((M, N), 12345.0, device="cuda",
                              dtype=torch.float32 if out == OUT_F32 else torch.bfloat16)
        Y = dmr.dmr_routed_linear(Xd, md, Wd, q, out, Y=sentinel.clone())
        Yl = dmr.dmr_lowbit_linear(Xd, q, out)
        Yh = dmr.dmr_dense_linear(Xd, Wd, out)
        mt = md.bool()
        assert torch.equal(Y[mt], Yh[mt])        # bit for bit, row by row
        assert torch.equal(Y[~mt], Yl[~mt])
    Y32 = dmr.dmr_routed_linear(Xd, md, Wd, q, OUT_F32).cpu().numpy().astype(np.float64)
    Yref = oracle.routed_linear(X, mask, W, *ref, bits=bits, group=group)
    assert rel_err(Y32, Yref) <= TOL
    return X, W, q, Y32


@pytest.mark.parametrize("kind", ["bernoulli", "all_low", "all_high", "alternating"])
@pytest.mark.parametrize("M", [4, 16, 64])
def test_routed_linear_masks(kind, M):
    if kind == "bernoulli":
        mask = inputs.precision_mask(M, 0.3, seed=11, index=M)
    elif kind == "all_low":
        mask = np.zeros(M, np.uint8)
    elif kind == "all_high":
        mask = np.ones(M, np.uint8)
    else:
        mask = (np.arange(M) % 2).astype(np.uint8) * 3   # any non-zero byte means high
    routed_case(M, 520, 640, 4, 128, mask)


def test_routed_linear_int8_and_ragged():
    mask = inputs.precision_mask(23, 0.5, seed=12)
    routed_case(23, 136, 384, 8, 0, mask)


@pytest.mark.parametrize("M,N,K", [(24, 1000, 4096), (31, 4096, 1024), (20, 22016, 512)])
def test_routed_rows_move_between_chunks(M, N, K):
    """17 to 32 rows run as chunks: a routed call moves rows from one chunk to another, and they must
    still come out bit for bit as in the unrouted call (every chunk uses the same kernel instance and summation
    order)."""
    mask = inputs.precision_mask(M, 0.4, seed=M)
    routed_case(M, N, K, 4, 128, mask)


@pytest.mark.parametrize("M", [12, 64])
def test_routed_calls_in_a_row_are_repeatable(M):
    """The two halves of a routed call run on two streams with scratch areas of their own; calls issued
    back to back on one workspace must keep giving the bits of the first call."""
    N, K = 1000, 4096
    W = inputs.weights(N, K, seed=31, index=M)
    X = inputs.activations(M, K, seed=31, index=M)
    q, _ = quantize_both(W, 4, 128)
    Xd, Wd = to_dev_bf16(X), to_dev_bf16(W)
    masks = [torch.from_numpy(inputs.precision_mask(M, p, seed=7, index=i)).cuda() for i, p in enumerate((0.3, 0.7, 0.0, 1.0))]
    ws = dmr.new_workspace(dmr.binding.OP_ROUTED, M, N, K, QFormat(4, 128), "cuda")
    first = [dmr.dmr_routed_linear(Xd, m, Wd, q, OUT_F32, workspace=ws).clone() for m in masks]
    for rep in range(15):
        outs = [dmr.dmr_routed_linear(Xd, m, Wd, q, OUT_F32, workspace=ws) for m in masks]
        for Yn, Y0 in zip(outs, first):
            assert torch.equal(Yn, Y0)


def test_routed_linear_prefill_sized_batch():
    # above 128 rows both the routed and the unrouted call take the persistent tensor-core kernel
    mask = inputs.precision_mask(300, 0.3, seed=15)
    routed_case(300, 264, 512, 4, 128, mask)


def test_routed_permutation_equivariance():
    M, N, K = 16, 264, 512
    mask = inputs.precision_mask(M, 0.4, seed=13)
    W = inputs.weights(N, K, seed=13)
    X = inputs.activations(M, K, seed=13)
    q = dmr.dmr_quantize(to_dev_bf16(W), QFormat(4, 128))
    Wd = to_dev_bf16(W)
    Y = dmr.dmr_routed_linear(to_dev_bf16(X), torch.from_numpy(mask).cuda(), Wd, q, OUT_F32)
    perm = np.random.default_rng(13).permutation(M)
    Yp = dmr.dmr_routed_linear(to_dev_bf16(X[perm]), torch.from_numpy(mask[perm]).cuda(), Wd, q, OUT_F32)
    assert torch.equal(Yp, Y[torch.from_numpy(perm).cuda()])


# ---------------- host-buffer entry point ----------------

def test_lowbit_linear_host_matches_device_call():
    M, N, K = 8, 520, 640
    W = inputs.weights(N, K, seed=14)
    X = inputs.activations(M, K, seed=14)
    q = dmr.dmr_quantize(to_dev_bf16(W), QFormat(4, 128))
    Xh = torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).pin_memory()
    Yh = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
    dmr.dmr_lowbit_linear_host(Xh, q, Yh, OUT_BF16)
    torch.cuda.synchronize()
    Yd = dmr.dmr_lowbit_linear(to_dev_bf16(X), q, OUT_BF16)
    assert torch.equal(Yh, Yd.cpu())


# ---------------- full-size shapes, sampled outputs ----------------

def test_decode_launch_chains_are_repeatable():
    """Back-to-back launches of the 4-bit decode kernel on one stream and one workspace (programmatic dependent
    launch lets a kernel start while its predecessor drains): every repetition must give the bits of the first one,
    and that one must match the oracle.  Layers with one to several tiles per CTA, 1-, 8- and 16-row batches.  (The
    streaming kernel's chains, with counters and partial sums in the workspace, are in test_gpu_full_size.py.)"""
    fmt = QFormat(4, 128)
    cases = []
    for (N, K, M) in [(3000, 11008, 1), (1024, 4096, 8), (3000, 11008, 16), (640, 2048, 16), (2200, 16384, 4)]:
        W = inputs.weights(N, K, seed=21, index=N + M)
        X = inputs.activations(M, K, seed=21, index=M + K)
        q, ref = quantize_both(W, 4, 128)
        Yref = oracle.lowbit_linear(X, *ref, bits=4, group=128)
        cases.append((to_dev_bf16(X), q, Yref, torch.empty((M, N), dtype=torch.float32, device="cuda")))
    ws = dmr.new_workspace(0, 16, 3000, 16384, fmt, "cuda")
    first = []
    for Xd, q, Yref, Y in cases:
        dmr.dmr_lowbit_linear(Xd, q, OUT_F32, Y=Y, workspace=ws)
        first.append(Y.clone())
        assert rel_err(Y.cpu().numpy().astype(np.float64), Yref) <= TOL_ROUNDED
    for rep in range(40):
        outs = []
        for Xd, q, Yref, Y in cases:
            Yn = torch.empty_like(Y)
            dmr.dmr_lowbit_linear(Xd, q, OUT_F32, Y=Yn, workspace=ws)
            outs.append(Yn)
        for Yn, Y0 in zip(outs, first):
            assert torch.equal(Yn, Y0)


@pytest.mark.parametrize("name,M", [("qkv", 1), ("o", 8), ("gate_up", 16), ("down", 16), ("gate_up", 4)])
def test_7b_decode_shapes_sampled(name, M):
    N, K = inputs.LAYER_7B[name]
    W = inputs.weights(N, K, seed=0, index=sorted(inputs.LAYER_7B).index(name))
    X = inputs.activations(M, K, seed=0, index=M)
    q, ref = quantize_both(W, 4, 128)
    assert_quant_equal(q, ref)
    Y32 = dmr.dmr_lowbit_linear(to_dev_bf16(X), q, OUT_F32).cpu().numpy().astype(np.float64)
    ms, ns = inputs.sample_outputs(M, N, 4000, seed=0)
    want = oracle.sampled_linear(X, ms, ns, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=4, group=128)
    # scale of the outputs from one fully computed row
    row = oracle.sampled_linear(X, np.zeros(N, np.int32), np.arange(N, dtype=np.int32),
                                qweight=ref[0], scales=ref[1], zeros=ref[2], bits=4, group=128)
    ymax = max(np.abs(row).max(), np.abs(want).max())
    assert np.abs(Y32[ms, ns] - want).max() / ymax <= TOL
    assert np.abs(Y32[0] - row).max() / ymax <= TOL
    assert np.isfinite(Y32).all()
