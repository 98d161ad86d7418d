"""Router calibration on the device against the oracle: the threshold bit for bit (binary64, same formula), the
mask byte for byte, and the mask fed straight into dmr_routed_linear."""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_02711_b200 as dmr
from paper_2602_02711_b200 import inputs, QFormat, OUT_F32
from helpers import to_dev_bf16

pytestmark = pytest.mark.gpu


def scores(n, seed, ties=False):
    rng = np.random.default_rng([seed, 77])
    x = rng.beta(2.0, 5.0, size=n).astype(np.float32)      # router scores: probabilities, most of them low
    if ties and n > 8:
        x[n // 2:n // 2 + 5] = x[0]
    return x


@pytest.mark.parametrize("n", [1, 2, 7, 256, 257, 3200, 65536])
@pytest.mark.parametrize("rho", [0.2, 0.4, 0.7, 0.0, 1.0])
def test_threshold_equals_the_oracle(n, rho):
    x = scores(n, n, ties=True)
    tau = dmr.dmr_router_calibrate(torch.from_numpy(x).cuda(), rho)
    assert float(tau[0].item()) == oracle.router_threshold(x, rho)


def test_mask_equals_the_oracle_and_meets_the_budget():
    cal = scores(3200, 5)
    for rho in (0.2, 0.4, 0.7):
        tau = dmr.dmr_router_calibrate(torch.from_numpy(cal).cuda(), rho)
        for M in (1, 64, 1000):
            p = scores(M, 100 + M)
            p[0] = np.float32(tau[0].item()) if np.float32(tau[0].item()) == tau[0].item() else p[0]
            mask = dmr.dmr_router_mask(torch.from_numpy(p).cuda(), tau).cpu().numpy()
            assert np.array_equal(mask, oracle.router_mask(p, oracle.router_threshold(cal, rho)))
        own = dmr.dmr_router_mask(torch.from_numpy(cal).cuda(), tau).cpu().numpy()
        assert abs(own.mean() - rho) <= 1.0 / len(cal) + 1e-12
    empty = dmr.dmr_router_mask(torch.zeros(0, dtype=torch.float32, device="cuda"), tau)
    assert empty.numel() == 0


def test_scores_to_routed_layer_without_leaving_the_device():
    M, N, K = 64, 520, 640
    W = inputs.weights(N, K, seed=51)
    X = inputs.activations(M, K, seed=51)
    cal, p = scores(3200, 6), scores(M, 7)
    tau = dmr.dmr_router_calibrate(torch.from_numpy(cal).cuda(), 0.4)
    mask_d = dmr.dmr_router_mask(torch.from_numpy(p).cuda(), tau)
    q = dmr.dmr_quantize(to_dev_bf16(W), QFormat(4, 128))
    Y = dmr.dmr_routed_linear(to_dev_bf16(X), mask_d, to_dev_bf16(W), q, OUT_F32).cpu().numpy().astype(np.float64)
    mask = oracle.router_mask(p, oracle.router_threshold(cal, 0.4))
    qw, sc, zp = oracle.quantize(W, bits=4, group=128)
    Yref = oracle.routed_linear(X, mask, W, qw, sc, zp, bits=4, group=128)
    assert 0 < mask.sum() < M
    assert np.abs(Y - Yref).max() / np.abs(Yref).max() <= 2e-3


def test_argument_errors():
    L = dmr.lib()
    x = torch.zeros(8, dtype=torch.float32, device="cuda")
    tau = torch.zeros(3, dtype=torch.float64, device="cuda")
    assert L.dmr_router_calibrate(x.data_ptr(), 0, 0.5, tau.data_ptr(), None) == 1
    assert L.dmr_router_calibrate(x.data_ptr(), 8, 1.5, tau.data_ptr(), None) == 1
    assert L.dmr_router_calibrate(x.data_ptr(), 70000, 0.5, tau.data_ptr(), None) == 2
    assert L.dmr_router_calibrate(None, 8, 0.5, tau.data_ptr(), None) == 1
