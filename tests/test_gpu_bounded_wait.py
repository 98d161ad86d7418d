"""A bounded wait that really runs out: the kernel returns, the status word says so, the context stays usable."""
import numpy as np
import pytest
import torch

import paper_2602_02711_b200 as dmr
from paper_2602_02711_b200 import inputs, QFormat, OUT_F32
from helpers import to_dev_bf16

pytestmark = pytest.mark.gpu

DMR_ERR_TIMEOUT = 6


def test_a_wait_nobody_answers_gives_up_and_reports():
    L = dmr.lib()
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    assert L.dmr_workspace_status(ws.data_ptr(), stream) == 0
    assert L.dmr_selftest_wait_timeout(ws.data_ptr(), ws.numel(), stream) == 0
    torch.cuda.synchronize()                                        # the kernel came back by itself
    words = ws.view(torch.int32).cpu().numpy()
    assert words[0] == DMR_ERR_TIMEOUT and words[1] == 2
    assert L.dmr_workspace_status(ws.data_ptr(), stream) == DMR_ERR_TIMEOUT
    assert b"wait" in L.dmr_status_string(DMR_ERR_TIMEOUT)
    # the context is intact: an ordinary call right afterwards works and leaves its own status word clean
    W = inputs.weights(64, 256, seed=3)
    X = inputs.activations(4, 256, seed=3)
    q = dmr.dmr_quantize(to_dev_bf16(W), QFormat(4, 128))
    ws2 = dmr.new_workspace(0, 4, 64, 256, QFormat(4, 128), "cuda")
    Y = dmr.dmr_lowbit_linear(to_dev_bf16(X), q, OUT_F32, workspace=ws2)
    assert np.isfinite(Y.cpu().numpy()).all()
    assert L.dmr_workspace_status(ws2.data_ptr(), stream) == 0


def test_selftest_rejects_a_missing_workspace():
    L = dmr.lib()
    assert L.dmr_selftest_wait_timeout(None, 0, None) == 4
