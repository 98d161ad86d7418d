"""The workspace-free entry point dmr_lowbit_linear_noalloc against dmr_lowbit_linear.

Some callers cannot allocate device memory at the moment they need a decode-time linear layer (a
serving loop whose memory all went to a cache pool at start-up, a plug-in that must not touch its
host's allocator). For them the library keeps the kernel's scratch in a fixed array of its own.
The array is shared by every call and keeps the previous call's contents, so the check runs two
calls back to back - with different shapes, so that the second meets the first one's leftovers -
and compares each with the ordinary entry point on the same inputs. This file is collected last.
"""
import numpy as np
import pytest
import torch

import paper_2602_02711_b200 as dmr
from paper_2602_02711_b200 import inputs, QFormat, OUT_BF16, OUT_F32
from helpers import to_dev_bf16

pytestmark = pytest.mark.gpu

TOL = 2e-3  # the bound the other linear-layer tests use; both calls run the same kernel, so they agree exactly


def one_case(M, N, K, bits, group, out, seed):
    W = inputs.weights(N, K, seed=seed, index=N)
    X = inputs.activations(M, K, seed=seed, index=M)
    q = dmr.dmr_quantize(to_dev_bf16(W), QFormat(bits, group))
    Xd = to_dev_bf16(X)
    want = dmr.dmr_lowbit_linear(Xd, q, out)                       # ordinary entry point, caller's workspace
    Y = torch.full((M, N), 777.0, device="cuda", dtype=torch.float32 if out == OUT_F32 else torch.bfloat16)
    dmr.dmr_lowbit_linear_noalloc(Xd, q, Y, out)                   # through the C ABI, no workspace
    torch.cuda.synchronize()
    a, b = Y.double().cpu().numpy(), want.double().cpu().numpy()
    assert np.abs(a - b).max() / np.abs(b).max() <= TOL
    assert torch.equal(Y, want)


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # first a layer whose feature groups are split across many CTAs (partial sums and counters in the
    # shared scratch), then a different shape and output type that reuses the same scratch
    one_case(8, 520, 4096, 4, 128, OUT_F32, seed=21)
    one_case(16, 1000, 1024, 4, 128, OUT_BF16, seed=22)


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
