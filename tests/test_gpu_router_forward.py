"""Parity of the router forward pass on the device (Sec. 4.1) with the float64 oracle, through the C ABI.

The kernels compute in fp32 with fused multiply-adds; against binary64 that leaves a few 1e-6 on the probabilities after
eight layers (rounding of sums of up to 1536 terms, renormalised by every layer norm).  Bar: max |p - p_ref| <= 2e-5.
A routing decision compares a probability with a threshold: decisions are compared where the oracle's probability is
further than that bar from the threshold, and the mask is required to be valid (0 / 1) everywhere.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_02711_b200 as dmr
from paper_2602_02711_b200 import inputs, RouterCfg

pytestmark = pytest.mark.gpu

TOL = 2e-5


def run(cfg_kw, B, L, seed, lengths=None):
    cfg = RouterCfg(**cfg_kw)
    p = inputs.router_params(**cfg_kw, seed=seed)
    Z = inputs.router_embeddings(B, L, cfg_kw["d"], seed=seed)
    n = inputs.router_lengths(B, L, seed=seed) if lengths is None else np.asarray(lengths, dtype=np.int32)
    want = oracle.router_forward(Z, n, p, cfg_kw["heads"])
    params = dmr.pack_router_params(p, cfg)
    probs, scores = dmr.dmr_router_forward(params, cfg, torch.from_numpy(Z).cuda(), torch.from_numpy(n).cuda(), score_class=1 if cfg_kw["classes"] > 1 else 0)
    got = probs.cpu().numpy().astype(np.float64)
    assert got.shape == want.shape
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= TOL
    assert np.abs(got.sum(axis=1) - 1.0).max() <= 1e-5
    col = 1 if cfg_kw["classes"] > 1 else 0
    assert torch.equal(scores, probs[:, col].contiguous())
    return got, want


@pytest.mark.parametrize("cfg_kw,B,L", [
    (dict(d=64, heads=4, ffn=128, layers=3, l_max=12, classes=3), 6, 9),          # small: several tiles of nothing, ragged everything
    (dict(d=384, heads=6, ffn=1536, layers=8, l_max=64, classes=2), 5, 33),       # the default depth at a sentence-encoder width
    (dict(d=384, heads=6, ffn=1536, layers=8, l_max=64, classes=2), 70, 17),      # more tokens than one row tile, T not a multiple of 64
    (dict(d=128, heads=1, ffn=64, layers=2, l_max=128, classes=1), 3, 128),       # one head of width 128, the longest sequence, one class
    (dict(d=1024, heads=16, ffn=1024, layers=1, l_max=8, classes=32), 2, 8),      # the widest model and the most classes
    (dict(d=48, heads=3, ffn=80, layers=16, l_max=5, classes=2), 9, 5),           # head width 16, deep
    (dict(d=384, heads=6, ffn=1536, layers=8, l_max=32, classes=2), 1, 32),       # one agent, one decision: the 32-token instance of the linears
    (dict(d=64, heads=4, ffn=128, layers=3, l_max=12, classes=3), 2, 8),          # 16 tokens
    (dict(d=64, heads=4, ffn=128, layers=3, l_max=12, classes=3), 1, 1),          # a single token
])
def test_router_forward_matches_oracle(cfg_kw, B, L):
    run(cfg_kw, B, L, seed=B + L)


def test_one_step_and_full_length_sequences():
    cfg_kw = dict(d=64, heads=2, ffn=128, layers=4, l_max=16, classes=2)
    run(cfg_kw, 4, 16, seed=3, lengths=[1, 1, 16, 16])


def test_padded_steps_never_matter_on_the_device():
    cfg_kw = dict(d=64, heads=4, ffn=128, layers=3, l_max=12, classes=2)
    cfg = RouterCfg(**cfg_kw)
    p = inputs.router_params(**cfg_kw, seed=8)
    params = dmr.pack_router_params(p, cfg)
    B, L = 4, 10
    Z = inputs.router_embeddings(B, L, 64, seed=8)
    n = np.array([1, 4, 7, 10], dtype=np.int32)
    Z2 = Z.copy()
    for b in range(B):
        Z2[b, n[b]:, :] = np.float32(1e6 * (b + 1))
    nd = torch.from_numpy(n).cuda()
    a, _ = dmr.dmr_router_forward(params, cfg, torch.from_numpy(Z).cuda(), nd)
    b2, _ = dmr.dmr_router_forward(params, cfg, torch.from_numpy(Z2).cuda(), nd)
    assert torch.equal(a, b2)
    # out-of-range lengths are clamped, never an out-of-bounds read
    c, _ = dmr.dmr_router_forward(params, cfg, torch.from_numpy(Z).cuda(), torch.tensor([0, 4, 7, 99], dtype=torch.int32).cuda())
    assert torch.equal(c, a)


def test_scores_feed_calibration_and_mask():
    # scores -> tau(rho) -> mask, all on the device, against the oracle's chain
    cfg_kw = dict(d=64, heads=4, ffn=128, layers=2, l_max=8, classes=2)
    cfg = RouterCfg(**cfg_kw)
    p = inputs.router_params(**cfg_kw, seed=9)
    B, L = 200, 8
    Z = inputs.router_embeddings(B, L, 64, seed=9)
    n = inputs.router_lengths(B, L, seed=9)
    probs, scores = dmr.dmr_router_forward(dmr.pack_router_params(p, cfg), cfg, torch.from_numpy(Z).cuda(), torch.from_numpy(n).cuda(), score_class=1)
    tau = dmr.dmr_router_calibrate(scores, 0.4)
    mask = dmr.dmr_router_mask(scores, tau).cpu().numpy()
    assert set(np.unique(mask)) <= {0, 1}
    want_p = oracle.router_forward(Z, n, p, 4)[:, 1]
    want_tau = oracle.router_threshold(want_p, 0.4)
    assert abs(float(tau[0].item()) - want_tau) <= TOL
    clear = np.abs(want_p - want_tau) > 2 * TOL
    assert np.array_equal(mask[clear], oracle.router_mask(want_p, want_tau)[clear])
    assert abs(mask.mean() - 0.4) <= 0.02


def test_router_forward_argument_errors():
    cfg = RouterCfg(d=64, heads=4, ffn=128, layers=1, l_max=8, classes=2)
    assert dmr.lib().dmr_router_param_floats(RouterCfg(d=60, heads=4, ffn=128, layers=1, l_max=8, classes=2)) == 0
    assert dmr.lib().dmr_router_param_floats(RouterCfg(d=64, heads=5, ffn=128, layers=1, l_max=8, classes=2)) == 0
    assert dmr.lib().dmr_router_workspace_bytes(cfg, 4, 9) == 0     # L beyond l_max
    n = dmr.lib().dmr_router_param_floats(cfg)
    assert n == 8 * 64 + (3 * 64 * 64 + 3 * 64 + 64 * 64 + 64 + 2 * 64 + 128 * 64 + 128 + 64 * 128 + 64 + 2 * 64) + 2 * 64 + 2
