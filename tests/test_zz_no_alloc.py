"""The workspace-free entry point dmr_lowbit_linear_noalloc against dmr_lowbit_linear and the oracle.

Some callers cannot allocate device memory at the moment they need a decode-time linear layer (a
serving loop whose memory all went to a cache pool at start-up, a plug-in that must not touch its
host's allocator). For them the library keeps the streaming kernel's scratch - feature-group counters,
per-CTA partial sums, a status word - in a fixed array of its own. The array is shared by every call
and keeps the previous call's contents, so the checks run calls back to back, with shapes large
enough that feature groups are split across CTAs (counters and partial sums really used) and with
widths that differ, so that one call meets the other's leftovers. This file is collected last.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_02711_b200 as dmr
from paper_2602_02711_b200 import inputs, QFormat, OUT_BF16, OUT_F32
from helpers import to_dev_bf16

pytestmark = pytest.mark.gpu

TOL = 2e-3        # the acceptance bound of the linear-layer tests
TOL_SUMS = 5e-5   # both entry points multiply exact integers; only the order of the fp32 sums differs


def prepare(M, N, K, bits, group, seed):
    W = inputs.weights(N, K, seed=seed, index=N)
    X = inputs.activations(M, K, seed=seed, index=M)
    q = dmr.dmr_quantize(to_dev_bf16(W), QFormat(bits, group))
    ref = oracle.quantize(W, bits=bits, group=group)
    ms, ns = inputs.sample_outputs(M, N, 2000, seed=seed)
    want = oracle.sampled_linear(X, ms, ns, qweight=ref[0], scales=ref[1], zeros=ref[2], bits=bits, group=group)
    return to_dev_bf16(X), q, (ms, ns, want)


def one_call(Xd, q, samples, out):
    M, N = Xd.shape[0], q.N
    want = dmr.dmr_lowbit_linear(Xd, q, out)                       # ordinary entry point, caller's workspace
    Y = torch.full((M, N), 777.0, device="cuda", dtype=torch.float32 if out == OUT_F32 else torch.bfloat16)
    dmr.dmr_lowbit_linear_noalloc(Xd, q, Y, out)                   # through the C ABI, no workspace
    torch.cuda.synchronize()
    a, b = Y.double().cpu().numpy(), want.double().cpu().numpy()
    scale = np.abs(b).max()
    assert np.isfinite(a).all()
    assert np.abs(a - b).max() / scale <= (TOL_SUMS if out == OUT_F32 else TOL)
    ms, ns, ref = samples
    assert np.abs(a[ms, ns] - ref).max() / scale <= (TOL_SUMS if out == OUT_F32 else 2 ** -8 + TOL)
    return Y


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # 8 x 8192 x 8192: 64 feature groups x 32 steps, far beyond what the cluster mode takes, so every CTA
    # shares feature groups with its neighbours through the counters and partial sums of the fixed array
    big = prepare(8, 8192, 8192, 4, 128, seed=21)
    small = prepare(16, 1000, 1024, 4, 128, seed=22)
    y0 = one_call(*big, OUT_F32)
    one_call(*small, OUT_BF16)            # a different shape and output type on the same scratch
    y1 = one_call(*big, OUT_F32)          # and the first one again: the array is as the first call found it
    assert torch.equal(y0, y1)


def test_layers_of_different_widths_share_the_scratch():
    # wide-then-narrow and narrow-then-wide: the counters of the wide layer's last feature groups must not be
    # where the narrow layer keeps partial sums
    wide = prepare(4, 13824, 5120, 4, 128, seed=24)
    narrow = prepare(4, 5120, 13824, 4, 128, seed=25)
    first = [one_call(*wide, OUT_F32), one_call(*narrow, OUT_F32)]
    for _ in range(3):
        assert torch.equal(one_call(*wide, OUT_F32), first[0])
        assert torch.equal(one_call(*narrow, OUT_F32), first[1])


def test_sizes_beyond_the_fixed_scratch_are_rejected():
    L = dmr.lib()
    assert L.dmr_noalloc_max_n() == 65536
    W = inputs.weights(64, 256, seed=23)
    q = dmr.dmr_quantize(to_dev_bf16(W), QFormat(4, 128))
    X = to_dev_bf16(inputs.activations(17, 256, seed=23))
    Y = torch.empty((17, 64), device="cuda", dtype=torch.bfloat16)
    with pytest.raises(dmr.DmrError) as e:
        dmr.dmr_lowbit_linear_noalloc(X, q, Y, OUT_BF16)           # M above the decode kernel's 16 rows
    assert e.value.code == 2
