"""Parity at the sizes and in the kernel instances the benchmark times.

The oracle cannot run these layers in full within seconds, so every case compares a few thousand seeded output
coordinates, one whole output row and one whole output column with oracle.sampled_linear (each output costs only K
multiply-adds), and asserts through dmr_describe_dispatch that the intended kernel instance is the one that ran:
the persistent prefill kernel with 256-row activation tiles and several tiles per CTA, the streaming kernel with
feature groups split across CTAs (no clusters) for bf16 and 8-bit weights, the 4-bit decode kernel, the routed call.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_02711_b200 as dmr
from paper_2602_02711_b200 import inputs, QFormat, OUT_BF16, OUT_F32
from paper_2602_02711_b200.binding import OP_LOWBIT, OP_DENSE
from helpers import to_dev_bf16, qweight_np, scales_np, zeros_np

pytestmark = pytest.mark.gpu

TOL = 2e-3
TOL_PREFILL = 3e-4   # one rounding of each dequantized weight to fp16
TOL_SUMS = 5e-5      # exact integer operands: only the order of the fp32 sums differs from the oracle


def sampled_reference(X, M, N, seed, count=3000, **layer):
    """(ms, ns, values) for seeded samples + row 0 + the last row + one column, and the scale of the outputs."""
    ms, ns = inputs.sample_outputs(M, N, count, seed=seed)
    col = int(ns[7]) if len(ns) > 7 else 0
    ms = np.concatenate([ms, np.zeros(N, np.int32), np.full(N, M - 1, np.int32), np.arange(M, dtype=np.int32)])
    ns = np.concatenate([ns, np.arange(N, dtype=np.int32), np.arange(N, dtype=np.int32), np.full(M, col, np.int32)])
    want = oracle.sampled_linear(X, ms, ns, **layer)
    return ms, ns, want, np.abs(want).max()


def check(Y, ms, ns, want, scale, tol):
    y = Y.double().cpu().numpy()
    assert np.isfinite(y).all()
    assert np.abs(y[ms, ns] - want).max() / scale <= tol


_layers = {}


def quantized_layer(N, K, bits, group, seed):
    """Seeded layer, quantized on the device and by the oracle (bit-exact), cached across the cases of this file."""
    key = (N, K, bits, group, seed)
    if key not in _layers:
        if len(_layers) >= 2:
            _layers.pop(next(iter(_layers)))
        W = inputs.weights(N, K, seed=seed, index=N + K)
        q = dmr.dmr_quantize(to_dev_bf16(W), QFormat(bits, group))
        ref = oracle.quantize(W, bits=bits, group=group)
        assert np.array_equal(qweight_np(q), ref[0]) and np.array_equal(scales_np(q), ref[1]) and np.array_equal(zeros_np(q), ref[2])
        _layers[key] = (W, q, ref)
    return _layers[key]


# ---------------- prefill: 7B-class shapes, the 256-row instance, several tiles per CTA ----------------

@pytest.mark.parametrize("name,M,bits,group", [
    ("o", 2048, 4, 128),       # 32 x 8 = 256 tiles of 128 x 256 on 148 CTAs
    ("qkv", 2048, 4, 128),     # 768 tiles: more than five per CTA
    ("qkv", 1900, 4, 128),     # M not a multiple of 256: a ragged last row tile
    ("o", 2048, 8, 0),         # INT8 per-channel
])
def test_prefill_7b_shapes(name, M, bits, group):
    N, K = inputs.LAYER_7B[name]
    plan = dmr.dmr_describe_dispatch(OP_LOWBIT, M, N, K, QFormat(bits, group))
    assert plan["kernel"] == "prefill" and plan["bn"] == 256 and plan["tiles"] > plan["ctas"]
    W, q, ref = quantized_layer(N, K, bits, group, seed=40)
    X = inputs.activations(M, K, seed=40, index=M)
    Xd = to_dev_bf16(X)
    Y32 = dmr.dmr_lowbit_linear(Xd, q, OUT_F32)
    ms, ns, want, scale = sampled_reference(X, M, N, 40, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=bits, group=group)
    check(Y32, ms, ns, want, scale, TOL_PREFILL)
    Y16 = dmr.dmr_lowbit_linear(Xd, q, OUT_BF16)
    assert torch.equal(Y16, Y32.to(torch.bfloat16))


def test_prefill_many_tiles_per_cta_with_ragged_features():
    # N not a multiple of 128 and M = 700: 3 row tiles x 44 feature tiles (the last one ragged), and a layer with
    # 1024 rows x 12288 features where every CTA runs two or three tiles back to back
    for (M, N, K) in [(700, 5600, 1024), (1024, 12288, 4096)]:
        plan = dmr.dmr_describe_dispatch(OP_LOWBIT, M, N, K, QFormat(4, 128))
        assert plan["kernel"] == "prefill" and plan["bn"] == 256
        W, q, ref = quantized_layer(N, K, 4, 128, seed=41)
        X = inputs.activations(M, K, seed=41, index=M)
        Y32 = dmr.dmr_lowbit_linear(to_dev_bf16(X), q, OUT_F32)
        ms, ns, want, scale = sampled_reference(X, M, N, 41, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=4, group=128)
        check(Y32, ms, ns, want, scale, TOL_PREFILL)
    assert dmr.dmr_describe_dispatch(OP_LOWBIT, 1024, 12288, 4096, QFormat(4, 128))["tiles"] >= 2 * 148


def test_prefill_split_k_over_two_row_tiles():
    # 300 rows = two 256-row tiles (the second ragged) x 32 feature tiles leave SMs idle: every tile's k range is split in
    # two work items, fp32 partial sums added in split order by the second kernel
    name, M = "down", 300
    N, K = inputs.LAYER_7B[name]
    plan = dmr.dmr_describe_dispatch(OP_LOWBIT, M, N, K, QFormat(4, 128))
    assert plan["kernel"] == "prefill" and plan["bn"] == 256 and plan["splits"] == 2 and plan["tiles"] == 64
    W, q, ref = quantized_layer(N, K, 4, 128, seed=40)
    X = inputs.activations(M, K, seed=44, index=M)
    Xd = to_dev_bf16(X)
    Y32 = dmr.dmr_lowbit_linear(Xd, q, OUT_F32)
    ms, ns, want, scale = sampled_reference(X, M, N, 44, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=4, group=128)
    check(Y32, ms, ns, want, scale, TOL_PREFILL)
    assert torch.equal(dmr.dmr_lowbit_linear(Xd, q, OUT_BF16), Y32.to(torch.bfloat16))
    assert torch.equal(dmr.dmr_lowbit_linear(Xd, q, OUT_F32), Y32)  # the sum order is fixed: repeatable bit for bit


@pytest.mark.parametrize("bits", [4, 3])
def test_prefill_64_row_tile_several_tiles_per_cta(bits):
    # up to 64 rows run the 64-row instance; 40000 features = 313 feature tiles (the last one ragged) on 148 CTAs,
    # no split along k: every CTA runs two or three tiles back to back through both accumulators
    M, N, K = 50, 40000, 1024
    plan = dmr.dmr_describe_dispatch(OP_LOWBIT, M, N, K, QFormat(bits, 128))
    assert plan["kernel"] == "prefill" and plan["bn"] == 64 and plan["splits"] == 1 and plan["tiles"] > 2 * plan["ctas"]
    W, q, ref = quantized_layer(N, K, bits, 128, seed=43)
    X = inputs.activations(M, K, seed=43, index=M)
    Y32 = dmr.dmr_lowbit_linear(to_dev_bf16(X), q, OUT_F32)
    ms, ns, want, scale = sampled_reference(X, M, N, 43, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=bits, group=128)
    check(Y32, ms, ns, want, scale, TOL_PREFILL)


# ---------------- streaming kernel with feature groups split across CTAs (no clusters) ----------------

@pytest.mark.parametrize("M,out", [(1, OUT_F32), (16, OUT_BF16), (27, OUT_F32)])
def test_dense_decode_contiguous_split(M, out):
    N, K = 2304, 8192     # 18 feature groups x 128 steps of 64 bf16 weights = 2304 steps
    plan = dmr.dmr_describe_dispatch(OP_DENSE, M, N, K)
    assert plan["kernel"] == "stream" and plan["cluster"] == 0 and plan["steps"] > 2100
    W = inputs.weights(N, K, seed=42, index=1)
    X = inputs.activations(M, K, seed=42, index=M)
    Xd, Wd = to_dev_bf16(X), to_dev_bf16(W)
    Y = dmr.dmr_dense_linear(Xd, Wd, out)
    ms, ns, want, scale = sampled_reference(X, M, N, 42, W=W)
    check(Y, ms, ns, want, scale, TOL_SUMS if out == OUT_F32 else 2 ** -8 + TOL_SUMS)
    assert torch.equal(dmr.dmr_dense_linear(Xd, Wd, out), Y)


@pytest.mark.parametrize("M,N,K,group,out", [
    (8, 4096, 8192, 0, OUT_F32),      # INT8 per-channel, 32 groups x 64 steps
    (16, 4096, 8192, 0, OUT_BF16),
    (32, 2048, 16384, 128, OUT_F32),  # INT8 grouped, the 32-row instance
])
def test_int8_decode_contiguous_split(M, N, K, group, out):
    plan = dmr.dmr_describe_dispatch(OP_LOWBIT, M, N, K, QFormat(8, group))
    assert plan["kernel"] == "stream" and plan["cluster"] == 0 and plan["steps"] > 1600
    W, q, ref = quantized_layer(N, K, 8, group, seed=43)
    X = inputs.activations(M, K, seed=43, index=M)
    Xd = to_dev_bf16(X)
    Y = dmr.dmr_lowbit_linear(Xd, q, out)
    ms, ns, want, scale = sampled_reference(X, M, N, 43, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=8, group=group)
    check(Y, ms, ns, want, scale, TOL_SUMS if out == OUT_F32 else 2 ** -8 + TOL_SUMS)
    assert torch.equal(dmr.dmr_lowbit_linear(Xd, q, out), Y)


def test_streaming_chain_on_one_workspace_is_repeatable():
    """bf16 and 8-bit layers of different widths, all split across CTAs, launched back to back on one workspace
    (programmatic dependent launch; counters and partial sums reused): every repetition gives the first bits."""
    shapes = [(2304, 8192, 16, 1), (4096, 8192, 8, 8), (4608, 4096, 16, 27), (2048, 16384, 8, 16)]   # N, K, bits, M
    cases = []
    for (N, K, bits, M) in shapes:
        X = to_dev_bf16(inputs.activations(M, K, seed=44, index=M))
        W = inputs.weights(N, K, seed=44, index=N)
        layer = to_dev_bf16(W) if bits == 16 else dmr.dmr_quantize(to_dev_bf16(W), QFormat(8, 0))
        op = OP_DENSE if bits == 16 else OP_LOWBIT
        plan = dmr.dmr_describe_dispatch(op, M, N, K, QFormat(8, 0))
        assert plan["kernel"] == "stream" and plan["cluster"] == 0
        Xb = inputs.activations(M, K, seed=44, index=M)
        if bits == 16:
            ref = sampled_reference(Xb, M, N, 44, count=500, W=W)
        else:
            r = oracle.quantize(W, bits=8, group=0)
            ref = sampled_reference(Xb, M, N, 44, count=500, qweight=r[0], scales=r[1], zeros=r[2], bits=8, group=0)
        cases.append((X, layer, bits, M, N, ref))
    ws = dmr.new_workspace(OP_LOWBIT, 32, 4608, 16384, QFormat(8, 0), "cuda")

    def run_all():
        outs = []
        for X, layer, bits, M, N, _ in cases:
            Y = torch.empty((M, N), dtype=torch.float32, device="cuda")
            if bits == 16:
                dmr.dmr_dense_linear(X, layer, OUT_F32, Y=Y, workspace=ws)
            else:
                dmr.dmr_lowbit_linear(X, layer, OUT_F32, Y=Y, workspace=ws)
            outs.append(Y)
        return outs

    first = run_all()
    for Y0, case in zip(first, cases):
        check(Y0, *case[5], TOL_SUMS)
    for _ in range(25):
        for Yn, Y0 in zip(run_all(), first):
            assert torch.equal(Yn, Y0)
    assert dmr.lib().dmr_workspace_status(ws.data_ptr(), torch.cuda.current_stream().cuda_stream) == 0


# ---------------- 4-bit decode kernel at 14B- and 32B-class sizes ----------------

@pytest.mark.parametrize("N,K,group,M,outlier", [
    (27648, 5120, 64, 1, 0.01),
    (27648, 5120, 64, 32, 0.01),
    (5120, 27648, 64, 16, 0.01),
    (5120, 27648, 64, 1, 0.01),
    (13824, 5120, 128, 8, 0.0),
])
def test_decode_w4_large_layers(N, K, group, M, outlier):
    plan = dmr.dmr_describe_dispatch(OP_LOWBIT, M, N, K, QFormat(4, group))
    assert plan["kernel"] == "decode_w4"
    W, q, ref = quantized_layer(N, K, 4, group, seed=45)
    X = inputs.activations(M, K, seed=45, index=M, outlier_frac=outlier)
    Y32 = dmr.dmr_lowbit_linear(to_dev_bf16(X), q, OUT_F32)
    ms, ns, want, scale = sampled_reference(X, M, N, 45, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=4, group=group)
    check(Y32, ms, ns, want, scale, TOL_SUMS)


@pytest.mark.parametrize("N,K,M", [(27648, 5120, 64), (5120, 27648, 256), (27648, 5120, 1)])
def test_int8_per_channel_32b_layers(N, K, M):
    W, q, ref = quantized_layer(N, K, 8, 0, seed=46)
    X = inputs.activations(M, K, seed=46, index=M, outlier_frac=0.01)
    Y32 = dmr.dmr_lowbit_linear(to_dev_bf16(X), q, OUT_F32)
    ms, ns, want, scale = sampled_reference(X, M, N, 46, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=8, group=0)
    check(Y32, ms, ns, want, scale, TOL_SUMS if M <= 32 else TOL_PREFILL)


@pytest.mark.parametrize("M", [64, 256])
def test_int4_g64_32b_layers_tensor_core_kernels(M):
    N, K = 27648, 5120
    W, q, ref = quantized_layer(N, K, 4, 64, seed=45)
    X = inputs.activations(M, K, seed=45, index=M, outlier_frac=0.01)
    Y32 = dmr.dmr_lowbit_linear(to_dev_bf16(X), q, OUT_F32)
    ms, ns, want, scale = sampled_reference(X, M, N, 45, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=4, group=64)
    check(Y32, ms, ns, want, scale, TOL_PREFILL)


# ---------------- routed batch on 14B-class linears ----------------

@pytest.mark.parametrize("name", ["k", "q", "gate"])
def test_routed_14b_linears(name):
    N, K = inputs.LAYER_14B[name]
    M = 64
    W, q, ref = quantized_layer(N, K, 4, 128, seed=47)
    X = inputs.activations(M, K, seed=47, index=M)
    mask = inputs.precision_mask(M, 0.3, seed=0)
    Xd, Wd, md = to_dev_bf16(X), to_dev_bf16(W), torch.from_numpy(mask).cuda()
    for out in (OUT_F32, OUT_BF16):
        Y = dmr.dmr_routed_linear(Xd, md, Wd, q, out)
        Yl = dmr.dmr_lowbit_linear(Xd, q, out)
        Yh = dmr.dmr_dense_linear(Xd, Wd, out)
        mt = md.bool()
        assert torch.equal(Y[mt], Yh[mt]) and torch.equal(Y[~mt], Yl[~mt])     # bit for bit, row by row
    Y32 = dmr.dmr_routed_linear(Xd, md, Wd, q, OUT_F32)
    ms, ns, want, scale = sampled_reference(X, M, N, 47, mask=mask, W=W, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=4, group=128)
    check(Y32, ms, ns, want, scale, TOL_PREFILL)
